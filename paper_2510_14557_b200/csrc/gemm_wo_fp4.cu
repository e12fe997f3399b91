// Weight-only GEMM for decode shapes on the FP4 tensor path, weights untouched by any thread:
//
//   D[M,N] = A(bf16)[M,K] * dec(W)[N,K]^T          (Sec. 7.1 setting; decode per Eq. 3)
//
// tcgen05.mma kind::mxf4 reads packed E2M1 codes with one E8M0 scale per 32 elements: exactly
// the stored form of the weights.  So the nibble plane goes from HBM to shared memory by plain
// TMA (128-byte rows of 256 codes, 128B swizzle) and from there into the tensor core.
//   * Every CTA (one per SM) owns a contiguous range of at most 128 weight rows and walks the
//     whole K with them: no split along K, no cross-CTA reduction; the rows of the 128-row MMA
//     tile it does not own are padding.
//   * The bf16 activations become FP4 as well: per block of 32, the magnitudes are cut into
//     seven base-4 digits (14 bits below the block's largest exponent), each digit plane an
//     operand row of E2M1 codes 0, 1, 2, 3 with its own block scale 2^(E - 1 - 2 j); the
//     epilogue adds the planes' accumulator columns.  An element within 2^6 of its block's
//     maximum is exact, a smaller one is rounded at 2^-14 of that maximum.
//   * MX+ weights: the tensor core reads the BM's code s m2 m1 m0 as the E2M1 value of its low
//     three bits instead of 4 + m/2 (Eq. 3).  Two threads per weight row add the difference,
//     (4 + m/2 - e2m1(m)) * 2^shared_exp * a[k_BM], on the CUDA cores: one multiply-add per block
//     and activation row, with the BM code read from the tile TMA wrote.
//   * Four warps turn the row-major scale bytes (TMA, 16 blocks per row at a time) into the
//     32-row x 16-byte atoms tcgen05.cp wants and drain the accumulators at the end; four more
//     issue the MMAs, each for every fourth stage with accumulators of its own (issuing one of
//     these small MMAs costs its thread tens of nanoseconds, whatever the MMA's size).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mxp {
namespace {

// warp 0: TMA producer; 1-4: MMA issuers; 5-8: row warps (scale atoms, epilogue); 9-20: BM
// correction (MX+ weights; otherwise they only help with the set-up).  (More issuers bought
// nothing, and past 672 threads the register allocation drops to 72 and the correction loop
// spills: with nearly all of the L1 given to shared memory a spill reload costs an L2 access.)
constexpr int kIssueWarp0 = 1, kIssuers = 4;
constexpr int kRowWarp0 = 5;
constexpr int kCorrWarp0 = 9, kCorrWarps = 12;
constexpr int kTpr = 4;              // correction threads per weight row
constexpr int kCorrRows = 32 * kCorrWarps / kTpr;  // weight rows per tile they can serve: 96
constexpr int kWarps = kCorrWarp0 + kCorrWarps;
constexpr int kThreads = 32 * kWarps;
constexpr int kStageK = 256;         // elements of K per stage: 128 bytes of codes per row
constexpr int kSlices = 7;           // base-4 digit planes of an activation
constexpr int kAcc = kIssuers;       // accumulators: one per issuer
constexpr uint32_t kTmemCols = 512;
constexpr int kAtom = 512;
constexpr int kMaxStages = 16;
constexpr int kMaxGroups = 32;       // groups of two stages (16 blocks) per tile: K <= 16384
// (the scale / index bytes of all groups of a tile are kept: the TMA thread never has to wait
// for a reader of theirs, in particular not for the activation set-up to finish)
// Activation rows per CTA: 1, 2 or 4.  The MMA's N is 16 (32 for 4): with one activation row its
// seven digit planes fill rows 0-6 and the tile pitch is 8 rows, so the MMA's rows 8-15 are the
// next stage's rows 0-7: finite E2M1 codes with finite scales whose accumulator columns nobody
// reads.  The scale atoms of the activations are kept at a pitch of their kN used rows.
__host__ __device__ constexpr int fp4_n(int ntok) { return ntok == 4 ? 32 : 16; }
__host__ __device__ constexpr int fp4_act_pitch(int ntok) { return ntok == 1 ? 1024 : fp4_n(ntok) * 128; }
__host__ __device__ constexpr int fp4_sfb_pitch(int ntok) { return fp4_n(ntok) * 16; }
constexpr long long kWaitLimit = 4000000000ll;
constexpr size_t kSmemMax = 227 * 1024;

struct Fp4Params {
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
struct Fp4Layout {
    size_t ring, ring_stride, sfa, meta, meta_stride, act, sfb, abf, corr, bars, total;
};
__host__ __device__ inline Fp4Layout fp4_layout(int K, int mrows, int rows_per_tile, int stages,
                                                bool plus, int ntok)
{
    Fp4Layout l;
    const size_t nst = (size_t)K / kStageK;
    const size_t rows8 = ((size_t)rows_per_tile + 7) / 8 * 8;
    size_t off = 0;
    l.ring = off;
    l.ring_stride = rows8 * 128;
    off += (size_t)stages * l.ring_stride;
    l.sfa = off;  // two atoms per stage of the tile: written once per tile
    off += nst * 2 * kAtom;
    l.meta = off;
    l.meta_stride = rows8 * 16 * (plus ? 2 : 1);  // scale tile, then (MX+) index tile
    off += (nst / 2) * l.meta_stride;
    off = (off + 1023) / 1024 * 1024;
    l.act = off;  // [stage][rows][128 bytes]; the last stage's MMA reads kN rows
    off += nst * (size_t)fp4_act_pitch(ntok) + (size_t)fp4_n(ntok) * 128;
    l.sfb = off;  // [stage][2 atoms]; the last copy reads a whole atom
    off += nst * 2 * (size_t)fp4_sfb_pitch(ntok) + kAtom;
    l.abf = off;
    if (plus) off += (size_t)mrows * (size_t)K * 2;
    off = (off + 15) / 16 * 16;
    l.corr = off;  // partial corrections [kTpr][ntok][128 rows], fp32
    if (plus) off += kTpr * (size_t)ntok * 128 * 4;
    l.bars = off;
    off += 1280;
    // the last slot's 128-row read must stay inside the allocation
    const size_t ring_read_end = l.ring + (size_t)(stages > 0 ? stages - 1 : 0) * l.ring_stride + 128 * 128;
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

#ifdef MXP_WOFP4_TIMELINE
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

// kTok: activation rows per CTA (1, 2 or 4; grid.y walks M); kPlus: the weights are MXFP4+.
template <int kTok, bool kPlus, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_wo_fp4_kernel(const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_sc,
                   const __grid_constant__ CUtensorMap tmap_ix, const Fp4Params prm)
{
    constexpr int kN = fp4_n(kTok);  // MMA N: kSlices * kTok digit rows, padded
    constexpr int kActPitch = fp4_act_pitch(kTok), kSfbPitch = fp4_sfb_pitch(kTok);
    static_assert(kSlices * kTok <= kN && kSlices * kTok <= kActPitch / 128, "digit rows must fit");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~(uintptr_t)1023);
    const int S = prm.stages;
    const int m0 = blockIdx.y * kTok;
    const int mrows = min(kTok, prm.M - m0);
    const Fp4Layout L = fp4_layout(prm.K, min(prm.M, kTok), prm.rows_per_tile, S, kPlus, kTok);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);  // TMA: weight tile landed
    uint64_t* empty = full + kMaxStages;       // MMAs (and BM reads) of the slot are done
    uint64_t* sfa_ready = empty + kMaxStages;  // [kMaxGroups] row warps wrote the group's scale atoms
    uint64_t* meta_full = sfa_ready + kMaxGroups;
    uint64_t* meta_empty = meta_full + kMaxGroups;
    uint64_t* acc_full = meta_empty + kMaxGroups;
    uint64_t* acc_empty = acc_full + 1;
    uint64_t* corr_full = acc_empty + 1;       // correction warps wrote their partial sums
    uint64_t* corr_empty = corr_full + 1;      // row warps have read them
    uint64_t* setup_bar = corr_empty + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(setup_bar + 1);
    volatile uint32_t* abort = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nb = prm.K / 32;
    const int nst = prm.K / kStageK;
    const int meta_bufs = nst / 2;  // one per group of two stages: all of a tile's
    const int rows8 = (prm.rows_per_tile + 7) / 8 * 8;

    auto ring = [&](int s) { return smem + L.ring + (size_t)s * L.ring_stride; };
    auto sfa = [&](int atom) { return smem + L.sfa + (size_t)atom * kAtom; };  // atom = 2 st + g
    auto meta_sc = [&](int g) { return smem + L.meta + (size_t)g * L.meta_stride; };
    auto meta_ix = [&](int g) { return smem + L.meta + (size_t)g * L.meta_stride + (size_t)rows8 * 16; };
    auto tile_n0 = [&](int t) {
        return ((int64_t)blockIdx.x * prm.tiles_per_cta + t) * prm.rows_per_tile;
    };

    // The set-up threads' first loads of the activations go out before anything else: their
    // latency is the longest single item of the prologue.
    const int ntask = nb * mrows * 4;  // four threads per block of 32 activations
    uint4 v_first = make_uint4(0u, 0u, 0u, 0u);
    if (warp != 0 && (int)threadIdx.x - 32 < ntask) {
        const int i = (int)threadIdx.x - 32, blk = i >> 2;
        const int kb = blk / mrows, mc = blk - kb * mrows;
        v_first = __ldg(reinterpret_cast<const uint4*>(prm.A + (int64_t)(m0 + mc) * prm.lda + kb * 32) + (i & 3));
    }
    if (threadIdx.x == 0) {
        TL(0);
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], kPlus ? 1 + kCorrWarps : 1);
        }
        for (int g = 0; g < kMaxGroups; ++g) ptx::mbar_init(&sfa_ready[g], 4);
        for (int g = 0; g < kMaxGroups; ++g) {
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
    const uint32_t tmem_acc = tmem_base;          // kAcc x kN columns (at most 256)
    const uint32_t tmem_sf = tmem_base + 256u;    // per issuer 16: per K group 4 for W, 4 for A

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
                    if ((st & 1) == 0) {
                        const int g = gc % meta_bufs;
                        const uint32_t ug = gc / meta_bufs;
                        if (ug > 0 && !ptx::mbar_wait(&meta_empty[g], (ug - 1) & 1, abort, kWaitLimit)) {
                            report(prm.status, abort, 0x6000 + g);
                            ok = false;
                            break;
                        }
                        ptx::mbar_arrive_expect_tx(&meta_full[g], meta_bytes);
                        ptx::tma_load_2d(meta_sc(g), &tmap_sc, &meta_full[g], (st >> 1) * 16, (int)n0);
                        if (kPlus)
                            ptx::tma_load_2d(meta_ix(g), &tmap_ix, &meta_full[g], (st >> 1) * 16, (int)n0);
                        ++gc;
                    }
                    const int s = c % S;
                    const uint32_t u = c / S;
                    if (u > 0 && !ptx::mbar_wait(&empty[s], (u - 1) & 1, abort, kWaitLimit)) {
                        report(prm.status, abort, 0x6100 + s);
                        ok = false;
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(&full[s], (uint32_t)prm.rows_per_tile * 128u);
                    ptx::tma_load_2d(ring(s), &tmap_w, &full[s], st * (kStageK / 2), (int)n0);
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- activations
        // bf16 -> seven planes of base-4 digits as E2M1 codes, each plane with its own E8M0
        // block scale: the MMA's K-major, 128B-swizzled narrow operand (row = plane * kTok +
        // activation row) plus the scale atoms; MX+ also keeps the bf16 values for the BM
        // correction.
        const int tid = threadIdx.x - 32;
        constexpr int kPrep = kThreads - 32;
        for (int i = tid; i < (nst * kActPitch + kN * 128) / 16; i += kPrep)   // absent rows: zero codes ...
            reinterpret_cast<uint4*>(smem + L.act)[i] = make_uint4(0u, 0u, 0u, 0u);
        for (int i = tid; i < (nst * 2 * kSfbPitch + kAtom) / 16; i += kPrep)  // ... with any finite scale
            reinterpret_cast<uint4*>(smem + L.sfb)[i] =
                make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);
        if (tid == 0) TL(70);
        asm volatile("bar.sync 1, %0;" ::"r"(kPrep) : "memory");  // the writes below land on top
        if (tid == 0) TL(71);
        // four threads per block of 32 activations, eight elements each
        for (int i0 = 0; i0 < ntask; i0 += kPrep) {
            const int i = i0 + tid;
            const bool on = i < ntask;
            const int blk = on ? i >> 2 : 0, qd = i & 3;
            const int kb = blk / mrows, mc = blk - kb * mrows;
            uint4 v = v_first;
            if (on) {
                if (i0 != 0)
                    v = __ldg(reinterpret_cast<const uint4*>(prm.A + (int64_t)(m0 + mc) * prm.lda + kb * 32) + qd);
                if (kPlus)
                    reinterpret_cast<uint4*>(smem + L.abf + ((size_t)mc * prm.K + kb * 32) * 2)[qd] = v;
            }
            const uint32_t x[4] = {v.x, v.y, v.z, v.w};
            // largest exponent field of the block (zero and subnormals count as field 1)
            uint32_t eb = 1;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                eb = max(eb, (x[q] >> 7) & 255u);
                eb = max(eb, (x[q] >> 23) & 255u);
            }
            eb = max(eb, __shfl_xor_sync(0xFFFFFFFFu, eb, 1));
            eb = max(eb, __shfl_xor_sync(0xFFFFFFFFu, eb, 2));
            if (tid == 0) TL(72);
            if (!on) continue;
            const bool nonfinite = eb == 255u;
            // 14-bit magnitude of an element relative to the block: |a| / 2^(E - 13)
            uint32_t qv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t h = (e & 1) ? x[e >> 1] >> 16 : x[e >> 1] & 0xFFFFu;
                const uint32_t ef = (h >> 7) & 255u;
                const uint32_t m8 = (ef ? 128u : 0u) | (h & 127u);
                const int sh = (int)max(ef, 1u) - (int)eb + 6;  // <= 6
                // (rounded to nearest when bits fall off the end: |error| <= 2^-15 of the block)
                const uint32_t mag = sh >= 0 ? m8 << sh : (sh > -9 ? (m8 + (1u << (-sh - 1))) >> (-sh) : 0u);
                qv[e] = mag | ((h >> 15) << 31);
            }
            uint8_t* tile = smem + L.act + (size_t)(kb >> 3) * kActPitch;
            uint32_t sgn = 0u;  // the eight sign bits, each on top of its nibble
#pragma unroll
            for (int e = 0; e < 8; ++e) sgn |= (qv[e] >> 31) << (4 * e + 3);
#pragma unroll
            for (int j = 0; j < kSlices; ++j) {
                const int sbyte = (int)eb - 1 - 2 * j;  // E8M0 byte of 2^(E - 1 - 2 j)
                uint32_t w = 0u;
                if (sbyte >= 0 && !nonfinite) {
                    // digit j of the eight elements, one per nibble ...
                    uint32_t d = 0u;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        constexpr int kDummy = 0;
                        (void)kDummy;
                        const int up = 4 * e - (12 - 2 * j);  // move bits 13-2j, 12-2j to nibble e
                        d |= (up >= 0 ? qv[e] << up : qv[e] >> (-up)) & (3u << (4 * e));
                    }
                    // ... as E2M1 codes: 0, 1, 2, 3 -> 000, 010, 100, 101 = 2 d - (d == 3); sign on top
                    w = ((d << 1) - ((d >> 1) & d & 0x11111111u)) | sgn;
                }
                const int row = j * kTok + mc;
                *reinterpret_cast<uint32_t*>(tile + swz_chunk((uint32_t)row, (uint32_t)(kb & 7)) + 4 * qd) = w;
                if (qd == 0)
                    smem[L.sfb + (size_t)(kb >> 2) * kSfbPitch + row * 16 + (kb & 3)] =
                        (uint8_t)(nonfinite ? 255 : max(sbyte, 0));
            }
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (threadIdx.x == 32) TL(2);
        if (lane == 0) ptx::mbar_arrive(setup_bar);
    }

    if (warp >= kIssueWarp0 && warp < kIssueWarp0 + kIssuers) {
        // ------------------------------------------------------------------ MMA issuers
        // Issuer i takes the stages st = i (mod kIssuers), with an accumulator and scale-factor
        // columns of its own.
        const int iss = warp - kIssueWarp0;
        bool ok = ptx::mbar_wait(setup_bar, 0, abort, kWaitLimit);
        if (!ok && lane == 0) report(prm.status, abort, 0x6200);
        if (lane == 0 && iss == 0) TL(3);
        ptx::tc_fence_after_sync();
        uint32_t c = 0, ti = 0;
        for (int t = 0; t < prm.tiles_per_cta && ok; ++t, ++ti) {
            if (tile_n0(t) >= prm.N) break;
            if (ti > 0 && !ptx::mbar_wait(acc_empty, (ti - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x6300);
                break;
            }
            ptx::tc_fence_after_sync();
            // stages are dealt out by their running number, so that slot and issuer stay paired
            // across tiles
            const int first = (iss - (int)(c % kIssuers) + kIssuers) % kIssuers;
            for (int st = first; st < nst; st += kIssuers) {
                const uint32_t cc = c + (uint32_t)st;
                const int s = cc % S;
                // (the number of slots is a multiple of kIssuers: an issuer sees every fill of
                // its slots in turn, so the parity of the fill it waits for is never ambiguous)
                if (!ptx::mbar_wait(&full[s], (cc / S) & 1, abort, kWaitLimit) ||
                    !ptx::mbar_wait(&sfa_ready[st >> 1], ti & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x6400 + s);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                if (lane == 0) TL(8 + st);
                const uint64_t da = ptx::smem_desc_sw128(ptx::smem_u32(ring(s)));
                const uint64_t db = ptx::smem_desc_sw128(ptx::smem_u32(smem + L.act + (size_t)st * kActPitch));
                if (ptx::elect_one()) {
#pragma unroll
                    for (int g = 0; g < 2; ++g) {  // 128 elements: one scale atom per operand
                        const uint32_t t_sfa = tmem_sf + 16u * (uint32_t)iss + 8u * (uint32_t)g;
                        const uint32_t t_sfb = t_sfa + 4u;
                        ptx::tc_cp_sf(t_sfa, ptx::smem_desc_sf(ptx::smem_u32(sfa(2 * st + g))));
                        ptx::tc_cp_sf(t_sfb, ptx::smem_desc_sf(ptx::smem_u32(
                                                 smem + L.sfb + (size_t)(2 * st + g) * kSfbPitch)));
#pragma unroll
                        for (int kk = 0; kk < 2; ++kk) {  // 64 elements = 32 bytes per MMA
                            const uint64_t adv = (uint64_t)((g * 2 + kk) * 32 >> 4);
                            ptx::mma_mxf4(tmem_acc + (uint32_t)(iss * kN), da + adv, db + adv,
                                          ptx::idesc_block_scaled(1, 1, 128, kN, 2 * kk, 2 * kk), t_sfa,
                                          t_sfb, (st == first && g == 0 && kk == 0) ? 0u : 1u);
                        }
                    }
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
            for (int st0 = 0; st0 < nst && ok; st0 += 2, ++gc) {
                const int g = gc % meta_bufs;
                if (!ptx::mbar_wait(&meta_full[g], (gc / meta_bufs) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x6600 + g);
                    ok = false;
                    break;
                }
                uint4 sc4 = make_uint4(0, 0, 0, 0);
                if (live) sc4 = *reinterpret_cast<const uint4*>(meta_sc(g) + row * 16);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&meta_empty[g]);
                if (live) {  // 16 blocks = two stages x two atoms, four blocks each
                    *reinterpret_cast<uint32_t*>(sfa(2 * st0) + sfa_off) = sc4.x;
                    *reinterpret_cast<uint32_t*>(sfa(2 * st0 + 1) + sfa_off) = sc4.y;
                    *reinterpret_cast<uint32_t*>(sfa(2 * st0 + 2) + sfa_off) = sc4.z;
                    *reinterpret_cast<uint32_t*>(sfa(2 * st0 + 3) + sfa_off) = sc4.w;
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&sfa_ready[st0 >> 1]);
            }
            if (!ok) break;
            // epilogue: every accumulator's digit-plane columns, plus the BM correction
            if (!ptx::mbar_wait_relaxed(acc_full, ti & 1, abort, kWaitLimit, 200u)) {
                if (lane == 0) report(prm.status, abort, 0x6900);
                break;
            }
            ptx::tc_fence_after_sync();
            if (threadIdx.x == 32 * kRowWarp0) TL(4);
            float acc[kN];
#pragma unroll
            for (int j = 0; j < kN; ++j) acc[j] = 0.f;
            for (int a = 0; a < kAcc; ++a) {
                // issuer a wrote its accumulator only if it had a stage of this tile
                if ((a - (int)((ti * (uint32_t)nst) % kIssuers) + kIssuers) % kIssuers >= nst) continue;
                uint32_t r2[kN];
                const uint32_t ta = tmem_acc + ((uint32_t)(32 * q) << 16) + (uint32_t)(a * kN);
                if (kN == 16)
                    ptx::tmem_ld_32x16(ta, reinterpret_cast<uint32_t(&)[16]>(r2[0]));
                else
                    ptx::tmem_ld_32x32(ta, reinterpret_cast<uint32_t(&)[32]>(r2[0]));
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < kN; ++j) acc[j] += __uint_as_float(r2[j]);
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty);
            float out[kTok];
#pragma unroll
            for (int m = 0; m < kTok; ++m) {
                out[m] = 0.f;
#pragma unroll
                for (int j = kSlices - 1; j >= 0; --j) out[m] += acc[j * kTok + m];  // small planes first
            }
            if (kPlus) {
                if (!ptx::mbar_wait_relaxed(corr_full, ti & 1, abort, kWaitLimit, 100u)) {
                    if (lane == 0) report(prm.status, abort, 0x6A00);
                    break;
                }
#pragma unroll
                for (int m = 0; m < kTok; ++m)
                    if (m < mrows)
                        for (int sub = 0; sub < kTpr; ++sub) out[m] += corr_s[(sub * kTok + m) * 128 + row];
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(corr_empty);
            }
            if (live) {
#pragma unroll
                for (int m = 0; m < kTok; ++m) {
                    if (m < mrows) {
                        const int64_t off = (int64_t)(m0 + m) * prm.ldd + n0 + row;
                        if (sizeof(OutT) == 4)
                            static_cast<float*>(prm.D)[off] = out[m];
                        else
                            static_cast<__nv_bfloat16*>(prm.D)[off] = __float2bfloat16_rn(out[m]);
                    }
                }
            }
        }
    } else if (kPlus && warp >= kCorrWarp0) {
        // ------------------------------------------------------------------ correction warps
        // Four threads per weight row, two blocks of each stage each: Eq. 3's BM value minus the
        // E2M1 value the tensor core read in its place, times the block's scale and the
        // activation at the BM's position.  Two stages (one group of scale / index bytes) are
        // taken together, so that four independent blocks are in flight per thread.
        const int tc = threadIdx.x - 32 * kCorrWarp0;
        const int row = tc >> 2, sub = tc & 3;
        const __nv_bfloat16* abf = reinterpret_cast<const __nv_bfloat16*>(smem + L.abf);
        float* corr_s = reinterpret_cast<float*>(smem + L.corr);
        uint32_t c = 0, gc = 0, ti = 0;
        bool ok = ptx::mbar_wait(setup_bar, 0, abort, kWaitLimit);  // the bf16 activations
        if (!ok && lane == 0) report(prm.status, abort, 0x6500);
        for (int t = 0; t < prm.tiles_per_cta && ok; ++t, ++ti) {
            const int64_t n0 = tile_n0(t);
            if (n0 >= prm.N) break;
            const int rows_here = (int)min((int64_t)prm.rows_per_tile, (int64_t)prm.N - n0);
            const bool live = row < rows_here;
            float corr[kTok];
#pragma unroll
            for (int m = 0; m < kTok; ++m) corr[m] = 0.f;
            for (int st0 = 0; st0 < nst && ok; st0 += 2, ++gc, c += 2) {
                const int g = gc % meta_bufs;
                const int s0 = c % S, s1 = (c + 1) % S;
                if (!ptx::mbar_wait(&meta_full[g], (gc / meta_bufs) & 1, abort, kWaitLimit) ||
                    !ptx::mbar_wait(&full[s0], (c / S) & 1, abort, kWaitLimit) ||
                    !ptx::mbar_wait(&full[s1], ((c + 1) / S) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x6800 + g);
                    ok = false;
                    break;
                }
                if (tc == 0) TL(40 + st0);
                if (live) {
                    // this thread's scale and index bytes: blocks 2 sub, 2 sub + 1 of either stage
                    const uint8_t* msc = meta_sc(g) + row * 16 + 2 * sub;
                    const uint8_t* mix = meta_ix(g) + row * 16 + 2 * sub;
                    const uint32_t scw = *reinterpret_cast<const uint16_t*>(msc) |
                                         ((uint32_t)*reinterpret_cast<const uint16_t*>(msc + 8) << 16);
                    const uint32_t ixw = *reinterpret_cast<const uint16_t*>(mix) |
                                         ((uint32_t)*reinterpret_cast<const uint16_t*>(mix + 8) << 16);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {  // stage u >> 1, block 2 sub + (u & 1)
                        const uint8_t* tile = ring((u >> 1) ? s1 : s0);
                        const uint32_t sc = (scw >> (8 * u)) & 255u;
                        const uint32_t e = 32u * (2u * (uint32_t)sub + (uint32_t)(u & 1)) + ((ixw >> (8 * u)) & 31u);
                        const uint32_t byte = tile[swz_chunk((uint32_t)row, e >> 5) + ((e & 31u) >> 1)];
                        const uint32_t nib = (e & 1u) ? byte >> 4 : byte & 15u;
                        // 2 * (4 + m/2 - e2m1(m)) for m = 0..7: 8 8 8 8 8 7 6 3
                        const uint32_t d2 = (0x36788888u >> (4u * (nib & 7u))) & 15u;
                        float v = (float)d2 * 0.5f * __uint_as_float(sc << 23);
                        if (nib & 8u) v = -v;
                        if (sc == 0u || sc == 255u) v = 0.f;  // flushed block / non-finite scale
                        const __nv_bfloat16* ap = abf + (size_t)(st0 + (u >> 1)) * kStageK + e;
#pragma unroll
                        for (int m = 0; m < kTok; ++m)
                            if (m < mrows) corr[m] = fmaf(v, __bfloat162float(ap[(size_t)m * prm.K]), corr[m]);
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    ptx::mbar_arrive(&meta_empty[g]);
                    ptx::mbar_arrive(&empty[s0]);
                    ptx::mbar_arrive(&empty[s1]);
                }
            }
            if (!ok) break;
            if (ti > 0 && !ptx::mbar_wait(corr_empty, (ti - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x6C00);
                break;
            }
            if (tc == 0) TL(60);
            if (row < 128) {
#pragma unroll
                for (int m = 0; m < kTok; ++m) corr_s[(sub * kTok + m) * 128 + row] = corr[m];
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(corr_full);
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncthreads();
    if (*abort != 0u && threadIdx.x == 0) {
        // after a timeout, copies may still be in flight into this CTA's shared memory: give
        // them (bounded) time to land before the CTA leaves
        const long long t0 = clock64();
        for (int s = 0; s < S; ++s)
            while (!ptx::mbar_try_wait(&full[s], 0) && !ptx::mbar_try_wait(&full[s], 1) &&
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

// Byte plane [rows][row_bytes]; boxes of box_bytes x box_rows, with or without the 128B swizzle.
bool make_tmap_bytes(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t row_bytes, int box_bytes,
                     int box_rows, bool swizzle)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Fp4Plan {
    int ntok, gx, mtiles, rows_per_tile, tiles_per_cta, stages;
    size_t smem;
};
// Rows per CTA so that every SM gets work, at most 128 per tile; as many ring slots as fit.
bool fp4_plan(int64_t M, int64_t N, int64_t K, bool plus, int num_sms, Fp4Plan* p)
{
    p->ntok = M <= 1 ? 1 : M <= 2 ? 2 : 4;
    p->mtiles = (int)((M + p->ntok - 1) / p->ntok);
    p->gx = num_sms / p->mtiles;
    if (p->gx < 1) p->gx = 1;
    const int64_t rows_per_cta = (N + p->gx - 1) / p->gx;
    const int max_rows = plus ? kCorrRows : 128;  // MX+: what the correction warps can serve
    p->tiles_per_cta = (int)((rows_per_cta + max_rows - 1) / max_rows);
    p->rows_per_tile = (int)((N + (int64_t)p->gx * p->tiles_per_cta - 1) / ((int64_t)p->gx * p->tiles_per_cta));
    const int mrows = (int)(M < p->ntok ? M : p->ntok);
    const size_t fixed = fp4_layout((int)K, mrows, p->rows_per_tile, 0, plus, p->ntok).total;
    const size_t per_stage = (size_t)((p->rows_per_tile + 7) / 8 * 8) * 128;
    if (fixed + 4 * per_stage + 128 * 128 > kSmemMax) return false;
    int stages = (int)((kSmemMax - fixed - 128 * 128) / per_stage);
    stages = stages > kMaxStages ? kMaxStages : stages;
    p->stages = stages / kIssuers * kIssuers;  // every slot belongs to one issuer
    p->smem = fp4_layout((int)K, mrows, p->rows_per_tile, p->stages, plus, p->ntok).total;
    return p->smem <= kSmemMax;
}

template <int kTok, bool kPlus, typename OutT>
cudaError_t launch(const CUtensorMap& tw, const CUtensorMap& ts, const CUtensorMap& ti, Fp4Params prm,
                   const Fp4Plan& plan, cudaStream_t stream)
{
    auto kern = gemm_wo_fp4_kernel<kTok, kPlus, OutT>;
    static SmemAttrOnce once;
    cudaError_t e = ensure_dynamic_smem(kern, (int)kSmemMax, once);
    if (e != cudaSuccess) return e;
    kern<<<dim3((unsigned)plan.gx, (unsigned)plan.mtiles), kThreads, plan.smem, stream>>>(tw, ts, ti, prm);
    return cudaGetLastError();
}

}  // namespace

bool wo_fp4_supported(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const mxp_packed& B)
{
    if (B.mode != MXP_MODE_MXFP4 && B.mode != MXP_MODE_MXFP4_PLUS) return false;
    if (M < 1 || M > 4 || N < 1 || N > (1ll << 30) || K < 512 || K % 512 != 0 || K > 8192) return false;
    if ((reinterpret_cast<uintptr_t>(A) & 15) || (reinterpret_cast<uintptr_t>(B.nibbles) & 15) ||
        (reinterpret_cast<uintptr_t>(B.scales) & 15))
        return false;
    if (B.mode != MXP_MODE_MXFP4 && (reinterpret_cast<uintptr_t>(B.bm_index) & 15)) return false;
    if (lda % 8 != 0) return false;
    const int sms = sm_count();
    Fp4Plan plan;
    return sms > 0 && fp4_plan(M, N, K, B.mode != MXP_MODE_MXFP4, sms, &plan);
}

cudaError_t launch_gemm_wo_fp4(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                               const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                               void* status, cudaStream_t stream)
{
    const bool plus = B.mode != MXP_MODE_MXFP4;
    const int sms = sm_count();
    Fp4Plan plan;
    if (sms <= 0 || !fp4_plan(M, N, K, plus, sms, &plan)) return cudaErrorNotSupported;
    // Decode calls come back with the same weights: the three tensor maps of the last weight
    // operand are kept (encoding them costs the host about as long as the kernel runs).
    struct MapKey {
        const void *nib, *sc, *ix;
        int64_t n, k;
        int rows, dev;
    };
    static std::mutex mu;
    static MapKey last = {};
    static CUtensorMap last_w, last_s, last_i;
    CUtensorMap tw, ts, ti;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        const MapKey key = {B.nibbles, B.scales, plus ? B.bm_index : B.scales, N, K, plan.rows_per_tile, dev};
        std::lock_guard<std::mutex> lock(mu);
        if (std::memcmp(&key, &last, sizeof(key)) != 0) {
            if (!make_tmap_bytes(&last_w, B.nibbles, N, K / 2, 128, plan.rows_per_tile, true) ||
                !make_tmap_bytes(&last_s, B.scales, N, K / 32, 16, plan.rows_per_tile, false) ||
                !make_tmap_bytes(&last_i, plus ? B.bm_index : B.scales, N, K / 32, 16, plan.rows_per_tile, false)) {
                last = MapKey{};
                return cudaErrorInvalidValue;
            }
            last = key;
        }
        tw = last_w;
        ts = last_s;
        ti = last_i;
    }
    Fp4Params prm;
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
#define MXP_FP4_LAUNCH(T, P)                                                  \
    (f32 ? launch<T, P, float>(tw, ts, ti, prm, plan, stream)                 \
         : launch<T, P, __nv_bfloat16>(tw, ts, ti, prm, plan, stream))
    if (plan.ntok == 1) return plus ? MXP_FP4_LAUNCH(1, true) : MXP_FP4_LAUNCH(1, false);
    if (plan.ntok == 2) return plus ? MXP_FP4_LAUNCH(2, true) : MXP_FP4_LAUNCH(2, false);
    return plus ? MXP_FP4_LAUNCH(4, true) : MXP_FP4_LAUNCH(4, false);
#undef MXP_FP4_LAUNCH
}

}  // namespace mxp
