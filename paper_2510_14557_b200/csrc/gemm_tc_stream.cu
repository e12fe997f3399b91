// Streamed CTA-pair GEMM on prepacked operands (sm_100a).
//
//   D[M,N] = dec(A)[M,K] * dec(B)[N,K]^T, fp32 accumulation in tensor memory.
//
// Everything the tensor core reads arrives in shared memory by TMA, so no thread touches
// operand data between HBM and the MMA.  That needs two cheap bandwidth passes first:
//
//   * scales: the row-major E8M0 plane is re-tiled into the 32-row x 16-byte atoms that
//     tcgen05.cp copies into tensor memory ([row group of 128][K group of 128][512 bytes]);
//   * MX+ operands (and their plain partner): every 4-bit code is widened to a 6-bit E2M3
//     code (sixteen of them in 12 bytes plus 4 bytes of padding: the form in which
//     kind::mxf8f6f4 reads 6-bit operands from shared memory).  E2M3 holds all E2M1 values and
//     the BM values 4 + m/2 of Eq. 3 exactly, so the block's BM is simply written as s 11 mmm
//     and one kind::mxf8f6f4 pass replaces the main MMA plus the residual MMAs of Eq. 4 /
//     Algorithm 1.  On this GPU such an MMA costs two FP4 MMAs, i.e. what one MX+ operand
//     costs with the split and half of what two cost.  (E4M3 bytes hold the same values and
//     cost the same tensor cycles, but more power: under the board's power limit the E2M3
//     form runs at a 4 % higher clock.  MX++ operands need E4M3's exponent range.)
//
// Plain MXFP4 x MXFP4 needs only the scale pass and runs kind::mxf4 on the nibble planes.
//
// One MXFP4+ operand against a plain MXFP4 one (the paper's main software scenario, Sec. 5:
// MXFP4+ activations, MXFP4 weights) keeps the FP4 rate for the main pass and adds Eq. 4's
// residual as a SPARSE MMA (Sec. 5.2, Algorithm 1): the MX+ operand is split once into
//   * its nibble plane with every BM's code replaced by BM_H (4 or 6, an E2M1 value), and
//   * BM_L (0, 0.5, 1 or 1.5 with the BM's sign; one value per block of 32, so the operand is
//     almost all zeros) stored 2:1 compressed with the metadata saying where each value sits.
// Per 128 elements of K the tensor core runs two dense kind::mxf4 instructions on the first
// and one sparse instruction (K = 128) on the second, into the same accumulator with the same
// scales: measured 1.5 times the plain MXFP4 issue time, against 2 times for the widened pass.
// The sparse operand has to be the instruction's A operand, so when the weights are the MX+
// side the kernel computes D^T = W A^T and its epilogue stores the tile transposed.
//
// Kernel: clusters of two CTAs, persistent, one 256 x 480 (kind::mxf4: 256 x 448) output tile
// per cluster and step, held in two accumulators that share the A tile: per flop that is 23 %
// fewer bytes through TMA than a 256 x 256 tile (kept for shapes whose larger tiles would fill
// the GPU unevenly).  Warp 0 of each CTA issues the TMA loads
// for its own 128 rows of A, its share of both halves of B and the scale atoms; all of them
// signal one mbarrier in the even CTA, whose warp 1 issues tcgen05.mma.cta_group::2 and commits
// to both CTAs.  Warps 2-9 drain the accumulators.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "e4m3_widen.cuh"

namespace mxp {

// ------------------------------------------------------------------------------ host helpers
EncodeFn tensormap_encode_fn()
{
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
                cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    });
    return fn;
}

int sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

// Output tile of a CTA pair: 256 rows x `halves` accumulators of sub_n() columns.  With two,
// they are 240 (kind::mxf4: 224) rather than 256 columns wide so that the scale factors (20
// tensor memory columns per K group in flight) fit beside them in the 512 columns.
constexpr int kTileM = 256;
constexpr int sub_n(bool wide, int halves) { return halves == 1 ? 256 : wide ? 240 : 224; }
constexpr int kRowBytes = 128;      // bytes of one operand row per stage (one swizzle span)
constexpr int kHalfTile = 128 * kRowBytes;  // 16 KB: this CTA's 128 rows of A
constexpr int kAtom = 512;          // scale bytes of 128 rows x 4 blocks
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr long long kWaitLimit = 4000000000ll;  // cycles (~2 s) before a wait gives up
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kFmtE4M3 = 0, kFmtE2M3 = 3;  // instruction-descriptor codes, kind::mxf8f6f4

// kWide = false: rows are 256 packed E2M1 codes (two scale atoms per stage), kind::mxf4.
// kWide = true : rows are 128 E2M3 / E4M3 code slots (one scale atom per stage), kind::mxf8f6f4.
// kHalves = 2: the tile has two halves (accumulators); 1: a single 256 x 256 accumulator, for
// shapes whose larger tiles would not fill the GPU evenly.
// kSparse (with kWide = false): A is an MXFP4+ operand split per Eq. 4; a stage also brings its
// compressed BM_L tile (64 bytes per row: 64-byte swizzle) and the sparsity metadata (16 bytes
// per row).
template <bool kWide, int kHalves, bool kSparse = false>
struct SCfg {
    static_assert(!(kWide && kSparse), "the sparse residual belongs to the FP4 path");
    static constexpr int kGroups = kWide ? 1 : 2;           // K groups of 128 elements per stage
    static constexpr int kSfA = kGroups * kAtom;            // own 128 rows of A
    static constexpr int kSubN = sub_n(kWide, kHalves);     // columns of one accumulator
    static constexpr int kTileN = kHalves * kSubN;
    static constexpr int kBRows = kSubN / 2;                // rows of a B half each CTA supplies
    static constexpr int kBTile = kBRows * kRowBytes;       // 15 (14) KB
    static constexpr int kSfB = 2 * kHalves * kGroups * kAtom;  // all rows of the B halves
    static constexpr int kRes = kSparse ? 128 * 64 : 0;     // compressed BM_L rows of this CTA
    static constexpr int kMeta = kSparse ? 128 * 16 : 0;    // their sparsity metadata
    static constexpr int kResOff = kHalfTile + kHalves * kBTile + kSfA + kSfB;  // multiple of 1024
    static constexpr int kStageRaw = kResOff + kRes + kMeta;
    static constexpr int kStage = (kStageRaw + 1023) / 1024 * 1024;  // swizzled tiles: 1024-aligned
    static constexpr int kStages = kSparse ? (kHalves == 2 ? 3 : 5) : (kHalves == 2 ? 4 : 6);
    static constexpr int kSmem = kStages * kStage + 1024 /*barriers*/ + 1024 /*align*/;
    static constexpr int kElemsPerStage = kWide ? 128 : 256;
};

struct SParams {
    int M, N, K;
    uint32_t a_fmt, b_fmt;  // kind::mxf8f6f4 operand formats (kFmtE2M3 / kFmtE4M3); wide only
    // An MXFP6+ operand is the sum of two E2M3 planes (its BM does not fit one E2M3 code):
    // plane p of A starts at row p * M of its widened copy (B: p * N), and the K loop runs once
    // per pair of planes: D = sum over (pa, pb) of A_pa * B_pb^T, same scales in every pass.
    int parts_a, parts_b;
    void* D;
    int64_t ldd;
    int d_vec_ok;
    int transposed;  // the tile is D^T: accumulator row r, column c belong at D[c][r]
    StatusBlock* status;
};

__device__ __forceinline__ void give_up(volatile uint32_t* abort, StatusBlock* st, uint32_t where)
{
    *abort = 1u;
    if (st != nullptr) {
        atomicCAS(&st->code, 0u, (uint32_t)MXP_ERR_TIMEOUT);
        st->where = where;
    }
}

// Tile order: bands of kBand tile rows, walked column by column, so that the tiles in flight
// at any time (one per CTA pair) cover a compact block of the output and their A and B
// panels stay resident in L2 instead of being re-streamed from HBM every wave.  (16 measured
// best on the 8192 x 28672 x 8192 prefill shape; 8 and 4 are within 3 %.)
#ifndef MXP_S_BAND
#define MXP_S_BAND 16
#endif
constexpr int kBand = MXP_S_BAND;
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn)
{
    const int per_band = kBand * tiles_n;
    const int band = tile / per_band;
    const int r = tile - band * per_band;
    const int h = min(kBand, tiles_m - band * kBand);  // height of this (maybe last) band
    tn = r / h;
    tm = band * kBand + (r - tn * h);
}

template <bool kWide, int kHalves, bool kSparse, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_stream_kernel(const __grid_constant__ CUtensorMap tmap_a,
                      const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_sfa,
                      const __grid_constant__ CUtensorMap tmap_sfb,
                      const __grid_constant__ CUtensorMap tmap_res,
                      const __grid_constant__ CUtensorMap tmap_meta, const SParams prm)
{
    using C = SCfg<kWide, kHalves, kSparse>;
    constexpr int S = C::kStages;
    constexpr int G = C::kGroups;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * C::kStage);
    uint64_t* full = bars;           // even CTA's copy is used: TMA bytes of both CTAs
    uint64_t* empty = bars + S;      // local: the MMAs that read the stage have completed
    uint64_t* acc_full = bars + 2 * S;       // local
    uint64_t* acc_empty = bars + 2 * S + 1;  // even CTA's copy: epilogue warps of both CTAs
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 2);
    volatile uint32_t* abort = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);

    auto a_tile = [&](int s) { return smem + s * C::kStage; };
    auto b_tile = [&](int s, int j) { return smem + s * C::kStage + kHalfTile + j * C::kBTile; };
    auto sfa = [&](int s) { return smem + s * C::kStage + kHalfTile + kHalves * C::kBTile; };
    auto sfb = [&](int s) { return smem + s * C::kStage + kHalfTile + kHalves * C::kBTile + C::kSfA; };
    auto res_tile = [&](int s) { return smem + s * C::kStage + C::kResOff; };
    auto meta_tile = [&](int s) { return smem + s * C::kStage + C::kResOff + C::kRes; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();  // 0: issues the MMAs
    const int kbase = (prm.K + C::kElemsPerStage - 1) / C::kElemsPerStage;  // stages of one pass
    const int kstages = kbase * prm.parts_a * prm.parts_b;
    const int tiles_m = (prm.M + kTileM - 1) / kTileM;
    const int tiles_n = (prm.N + C::kTileN - 1) / C::kTileN;
    const int num_tiles = tiles_m * tiles_n;
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 1);
        }
        ptx::mbar_init(acc_full, 1);
        ptx::mbar_init(acc_empty, 2 * kEpiWarps);
        *abort = 0u;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_a);
        ptx::prefetch_tmap(&tmap_b);
        ptx::prefetch_tmap(&tmap_sfa);
        ptx::prefetch_tmap(&tmap_sfb);
        if (kSparse) {
            ptx::prefetch_tmap(&tmap_res);
            ptx::prefetch_tmap(&tmap_meta);
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc_2cta(tmem_slot, kTmemCols);
        ptx::tmem_relinquish_2cta();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // both CTAs' barriers exist before anything signals them remotely
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    ClockStamp* stamp = reinterpret_cast<ClockStamp*>(reinterpret_cast<uint8_t*>(prm.status) +
                                                      kClockStampOffset);
#ifdef MXP_S_GRIDSTAMP  // measurement builds: earliest begin, latest and earliest end over all CTAs
    if (threadIdx.x == 64) atomicMin(reinterpret_cast<unsigned long long*>(stamp) + 4, ptx::globaltimer_ns());
#endif
    // Accumulators at columns 0 and 256; scale factors in the gaps behind them.  Per K group:
    // 4 columns for A's 128 rows, 8 for each half of B.  Two halves: kind::mxf8f6f4 has one
    // group in flight (A at 240, B halves at 248 and 496); kind::mxf4 two (group g at
    // 224 + 256 g: A, then the B halves 8 and 16 columns on).  One half: A at 256 + 4 g, B at
    // 264 + 8 g.
    auto tmem_sfa = [&](int g) {
        return tmem_base + (kHalves == 1 ? 256u + 4u * g : kWide ? 240u : 224u + 256u * g);
    };
    auto tmem_sfb = [&](int g, int j) {
        return tmem_base + (kHalves == 1 ? 264u + 8u * g
                            : kWide      ? (j == 0 ? 248u : 496u)
                                         : 232u + 256u * g + 8u * j);
    };
    // Sparsity metadata of a stage: four columns (two per K group) behind the scale factors
    // (two halves: group 0's occupy columns 224..247; one half: 256..279).
    const uint32_t tmem_meta = tmem_base + (kHalves == 1 ? 288u : 248u);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t full0 = ptx::map_to_cta(ptx::smem_u32(&full[0]), 0);
            // the launch may overlap the tail of the prepack kernel: its output is first
            // touched here
            ptx::grid_dependency_wait();
            if (blockIdx.x == 0) {  // the kernel's own work starts here: what came before is the
                                    // tail of the grid it depends on
                stamp->clk_begin = (unsigned long long)clock64();
                stamp->ns_begin = ptx::globaltimer_ns();
            }
            uint32_t c = 0;
            bool ok = true;
            // Bytes the barrier of a stage sees from both CTAs' copies.  E2M3 operands lie packed in
            // global memory, 12 bytes per 16 codes, and the copy spreads them into 16-byte slots:
            // the barrier counts the 12.
            const uint32_t stage_tx =
                2u * (uint32_t)(C::kStageRaw - ((kWide && prm.a_fmt == kFmtE2M3) ? kHalfTile / 4 : 0) -
                                ((kWide && prm.b_fmt == kFmtE2M3) ? kHalves * C::kBTile / 4 : 0));
            for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
                int tm, tn;
                tile_coords(tile, tiles_m, tiles_n, tm, tn);
                const int m0 = tm * kTileM + 128 * (int)rank;
                const int n0 = tn * C::kTileN + C::kBRows * (int)rank;
                int kk = 0, pa = 0, pb = 0;  // stage within the pass, plane of A, plane of B
                for (int kt = 0; kt < kstages; ++kt, ++c) {
                    const int s = c % S;
                    const uint32_t use = c / S;
                    const int ka = kk, ya = pa * prm.M, yb = pb * prm.N;
                    if (++kk == kbase) {
                        kk = 0;
                        if (++pb == prm.parts_b) {
                            pb = 0;
                            ++pa;
                        }
                    }
                    if (use > 0 && !ptx::mbar_wait(&empty[s], (use - 1) & 1, abort, kWaitLimit)) {
                        give_up(abort, prm.status, 0x2100 + s);
                        ok = false;
                        break;
                    }
                    if (rank == 0) ptx::mbar_arrive_expect_tx(&full[s], stage_tx);
                    ptx::tma_load_2d_pair(a_tile(s), &tmap_a, full0 + 8u * (uint32_t)s, ka * kRowBytes, ya + m0);
#pragma unroll
                    for (int j = 0; j < kHalves; ++j)
                        ptx::tma_load_2d_pair(b_tile(s, j), &tmap_b, full0 + 8u * (uint32_t)s,
                                              ka * kRowBytes, yb + n0 + j * C::kSubN);
                    ptx::tma_load_3d_pair(sfa(s), &tmap_sfa, full0 + 8u * (uint32_t)s, 0, ka * G, 2 * tm + (int)rank);
                    ptx::tma_load_3d_pair(sfb(s), &tmap_sfb, full0 + 8u * (uint32_t)s, 0, ka * G,
                                          2 * kHalves * tn);
                    if (kSparse) {
                        ptx::tma_load_2d_pair(res_tile(s), &tmap_res, full0 + 8u * (uint32_t)s, ka * 64, m0);
                        ptx::tma_load_3d_pair(meta_tile(s), &tmap_meta, full0 + 8u * (uint32_t)s, 0, ka * 4,
                                              2 * tm + (int)rank);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (rank == 0) {
            uint32_t c = 0, ti = 0;
            bool ok = true;
            for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++ti) {
                int tm, tn;
                tile_coords(tile, tiles_m, tiles_n, tm, tn);
                // a right half that lies wholly past column N gets no MMAs
                const int halves = (kHalves == 2 && tn * C::kTileN + C::kSubN < prm.N) ? 2 : 1;
                if (ti > 0 &&
                    !ptx::mbar_wait_cluster(acc_empty, (ti - 1) & 1, abort, kWaitLimit)) {
                    if (lane == 0) give_up(abort, prm.status, 0x2600);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                uint32_t accumulate = 0;
                for (int kt = 0; kt < kstages && ok; ++kt, ++c) {
                    const int s = c % S;
                    const uint32_t ph = (c / S) & 1;
                    if (!ptx::mbar_wait(&full[s], ph, abort, kWaitLimit)) {
                        if (lane == 0) give_up(abort, prm.status, 0x2200 + s);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint64_t da = ptx::smem_desc_sw128(ptx::smem_u32(a_tile(s)));
                    const uint64_t d_sfa = ptx::smem_desc_sf(ptx::smem_u32(sfa(s)));
                    const uint64_t d_sfb = ptx::smem_desc_sf(ptx::smem_u32(sfb(s)));
                    const int groups =
                        kWide ? 1 : ((prm.K - (kt % kbase) * C::kElemsPerStage) >= C::kElemsPerStage ? 2 : 1);
                    if (ptx::elect_one()) {
                        for (int g = 0; g < groups; ++g) {
                            ptx::tc_cp_sf_2cta(tmem_sfa(g), d_sfa + (uint64_t)(kAtom * g >> 4));
                            // B's atoms in shared memory: [half j][128-row part h][K group g]
#pragma unroll
                            for (int jh = 0; jh < 2 * kHalves; ++jh)
                                ptx::tc_cp_sf_2cta(tmem_sfb(g, jh >> 1) + 4 * (jh & 1),
                                                   d_sfb + (uint64_t)((G * kAtom * jh + kAtom * g) >> 4));
                            if (kSparse && g == 0)
                                ptx::tc_cp_128x128b_2cta(tmem_meta, ptx::smem_desc_sf(ptx::smem_u32(meta_tile(s))));
                            for (int j = 0; j < halves; ++j) {
                                const uint32_t tmem_acc = tmem_base + 256u * j;
                                const uint64_t db = ptx::smem_desc_sw128(ptx::smem_u32(b_tile(s, j)));
                                if (kWide) {
#pragma unroll
                                    for (int kk = 0; kk < 4; ++kk) {
                                        const uint32_t idesc = ptx::idesc_block_scaled(
                                            prm.a_fmt, prm.b_fmt, kTileM, C::kSubN, kk, kk);
                                        ptx::mma_mxf8f6f4_2cta(tmem_acc, da + (uint64_t)(2 * kk),
                                                               db + (uint64_t)(2 * kk), idesc,
                                                               tmem_sfa(g), tmem_sfb(g, j),
                                                               accumulate | (uint32_t)kk);
                                    }
                                } else {
#pragma unroll
                                    for (int kk = 0; kk < 2; ++kk) {
                                        const uint64_t adv = (uint64_t)((g * 2 + kk) * 32 >> 4);
                                        const uint32_t idesc = ptx::idesc_block_scaled(
                                            1, 1, kTileM, C::kSubN, 2 * kk, 2 * kk);
                                        ptx::mma_mxf4_2cta(tmem_acc, da + adv, db + adv, idesc,
                                                           tmem_sfa(g), tmem_sfb(g, j),
                                                           accumulate | (uint32_t)(g | kk));
                                    }
                                    if (kSparse) {
                                        // Eq. 4's BM_L term over the same 128 elements of K: 32
                                        // bytes of compressed A per row, 64 bytes of B, all four
                                        // scale bytes of either operand's column
                                        const uint64_t dr =
                                            ptx::smem_desc_sw64(ptx::smem_u32(res_tile(s))) + (uint64_t)(2 * g);
                                        const uint32_t idesc =
                                            ptx::idesc_block_scaled(1, 1, kTileM, C::kSubN, 0, 0) | ptx::kIdescSparse;
                                        ptx::mma_sp_mxf4_2cta(tmem_acc, dr, db + (uint64_t)(4 * g),
                                                              tmem_meta + 2u * (uint32_t)g, idesc, tmem_sfa(g),
                                                              tmem_sfb(g, j), 1u);
                                    }
                                }
                            }
                        }
                        ptx::tc_commit_2cta(&empty[s]);
                    }
                    __syncwarp();
                    accumulate = 1;
                }
                if (ok) {
                    if (ptx::elect_one()) ptx::tc_commit_2cta(acc_full);
                    __syncwarp();
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        // Each warp owns 32 rows (its TMEM lane quarter) and moves chunks of half an accumulator
        // (120, 112 or 128 columns) through registers.  Two halves: warps 2-5 drain the left
        // accumulator, 6-9 the right one, two chunks each.  One half: warps 2-5 take its left
        // chunk, 6-9 its right chunk.
        // A warp releases the accumulators as soon as it has read its last chunk.
        const int q = warp & 3;  // the TMEM lane quarter this warp may read
        const int wsel = (warp - 2) >> 2;
        const int j = kHalves == 2 ? wsel : 0;
        const int ch0 = kHalves == 2 ? 0 : wsel, ch1 = kHalves == 2 ? 2 : wsel + 1;
        constexpr int kCols = C::kSubN / 2;
        const uint32_t acc_empty0 = ptx::map_to_cta(ptx::smem_u32(acc_empty), 0);
        uint32_t ti = 0;
        bool ok = true;
        for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++ti) {
            int tm, tn;
            tile_coords(tile, tiles_m, tiles_n, tm, tn);
            const int m0 = tm * kTileM + 128 * (int)rank, n0 = tn * C::kTileN + j * C::kSubN;
            if (!ptx::mbar_wait(acc_full, ti & 1, abort, kWaitLimit)) {
                give_up(abort, prm.status, 0x2500);
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            const int row = m0 + 32 * q + lane;
            const uint32_t taddr = tmem_base + 256u * j + ((uint32_t)(32 * q) << 16);
            for (int ch = ch0; ch < ch1; ++ch) {
                uint32_t rr[kCols];
                const uint32_t ta = taddr + ch * kCols;
                constexpr int k32 = kCols / 32, k16 = (kCols % 32) / 16, k8 = (kCols % 16) / 8;
#pragma unroll
                for (int cb = 0; cb < k32; ++cb)
                    ptx::tmem_ld_32x32(ta + 32 * cb, reinterpret_cast<uint32_t(&)[32]>(rr[32 * cb]));
                if (k16) ptx::tmem_ld_32x16(ta + 32 * k32, reinterpret_cast<uint32_t(&)[16]>(rr[kCols - 16 - 8 * k8]));
                if (k8) ptx::tmem_ld_32x8(ta + kCols - 8, reinterpret_cast<uint32_t(&)[8]>(rr[kCols - 8]));
                ptx::tmem_ld_wait();
                if (ch == ch1 - 1) {
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(acc_empty0);
                }
                const int col0 = n0 + ch * kCols;
                if (row >= prm.M || col0 >= prm.N) continue;
                if (kSparse && prm.transposed) {
                    // D[col][row]: a register holds one column of the tile, the warp's lanes
                    // hold 32 consecutive rows, i.e. 32 consecutive elements of a row of D
                    OutT* dcol = static_cast<OutT*>(prm.D) + (int64_t)col0 * prm.ldd + row;
#pragma unroll
                    for (int i = 0; i < kCols; ++i) {
                        if (col0 + i < prm.N) {
                            if (sizeof(OutT) == 4)
                                reinterpret_cast<float*>(dcol)[(int64_t)i * prm.ldd] = __uint_as_float(rr[i]);
                            else
                                reinterpret_cast<__nv_bfloat16*>(dcol)[(int64_t)i * prm.ldd] =
                                    __float2bfloat16_rn(__uint_as_float(rr[i]));
                        }
                    }
                    continue;
                }
                OutT* drow = static_cast<OutT*>(prm.D) + (int64_t)row * prm.ldd + col0;
                if (col0 + kCols <= prm.N && prm.d_vec_ok) {
                    uint4* p = reinterpret_cast<uint4*>(drow);
                    if (sizeof(OutT) == 4) {
#pragma unroll
                        for (int i = 0; i < kCols / 4; ++i)
                            p[i] = make_uint4(rr[4 * i], rr[4 * i + 1], rr[4 * i + 2], rr[4 * i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < kCols / 8; ++i) {
                            uint32_t o[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const __nv_bfloat162 h2 =
                                    __floats2bfloat162_rn(__uint_as_float(rr[8 * i + 2 * k]),
                                                          __uint_as_float(rr[8 * i + 2 * k + 1]));
                                o[k] = *reinterpret_cast<const uint32_t*>(&h2);
                            }
                            p[i] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kCols; ++i) {
                        if (col0 + i < prm.N) {
                            if (sizeof(OutT) == 4)
                                reinterpret_cast<float*>(drow)[i] = __uint_as_float(rr[i]);
                            else
                                reinterpret_cast<__nv_bfloat16*>(drow)[i] =
                                    __float2bfloat16_rn(__uint_as_float(rr[i]));
                        }
                    }
                }
            }
        }
    }

    if (blockIdx.x == 0 && threadIdx.x == 64) {
        stamp->clk_end = (unsigned long long)clock64();
        stamp->ns_end = ptx::globaltimer_ns();
    }
#ifdef MXP_S_GRIDSTAMP
    if (threadIdx.x == 64) {
        atomicMax(reinterpret_cast<unsigned long long*>(stamp) + 5, ptx::globaltimer_ns());
        atomicMin(reinterpret_cast<unsigned long long*>(stamp) + 6, ptx::globaltimer_ns());
    }
#endif
    // ---------------------------------------------------------------------- teardown
    // After a timeout, copies may still be in flight into this pair's shared memory: give
    // them (bounded) time to land before the CTAs leave.  `full` of the even CTA counts both.
    if (*abort != 0u && threadIdx.x == 0 && rank == 0) {
        const long long t0 = clock64();
        for (int s = 0; s < S; ++s)
            while (!ptx::mbar_try_wait(&full[s], 0) && !ptx::mbar_try_wait(&full[s], 1) &&
                   clock64() - t0 < kWaitLimit) {
            }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    // neither CTA may leave (or free its TMEM) while the other still reads its shared memory
    // through the pair MMA or signals its barriers
    ptx::cluster_sync();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_2cta(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------ prepack
// One launch prepares both operands.  Its CTAs are of two kinds, told apart by block index:
//
// scale CTAs: scale plane [rows][nbk] -> atoms [row groups][nbk/4][512]; inside an atom the
//   four scale bytes of row r (r < 128) sit at (r % 32) * 16 + (r / 32) * 4.  Row groups follow
//   the GEMM's accumulators: two per `tile_rows` rows (256 for A; 240 or 224, one half tile,
//   for B), the second starting 128 rows in, so for B it holds 112 or 96 rows.  Rows past the
//   end of the half tile or of the operand are written as zero.  A CTA handles one row group x up to 32 K groups
//   through shared memory, so reads and writes are both contiguous.
// widen CTAs (only when an operand is MX+): packed codes [rows][K/2] -> 16 bytes per 16 codes,
//   one thread per 16 elements (8 bytes in, 16 bytes out, both contiguous across the warp).
//   MXFP4 / MXFP4+: E2M3 codes, the E2M1 code with two zero mantissa bits appended, the BM of
//   an MX+ block (Eq. 3: 4 + m/2, stored as sign + 3 mantissa bits) as s 11 mmm; sixteen codes
//   packed into 12 bytes, 4 bytes of padding.  MX++: E4M3 bytes (E2M1 magnitudes 0, .5, 1, 1.5,
//   2, 3, 4, 6 are 00 30 38 3C 40 44 48 4C, the BM 0x48 | m, both rescaled by powers of two).
//   A block with scale byte 0 (flushed) becomes zeros.
struct PrepackOperand {
    const uint8_t* nibbles;
    const uint8_t* scales;
    const uint8_t* bm_index;  // nullptr: plain MXFP4
    uint8_t* atoms;
    uint8_t* wide;            // nullptr: not widened
    int rows, nbk;
    int tile_rows;            // rows per accumulator: kTileM for A, sub_n() for B
    int pp;                   // MX++ operand: index bits 7:5 hold delta (Sec. 4.3)
    int six;                  // source codes are packed 6-bit E2M3 (MXFP6 / MXFP6+), not nibbles
    int eight;                // source codes are E4M3 bytes (MXFP8): the MMA reads them as they are
    int eight_plus;           // MXFP8+: E4M3 bytes whose BM is an E0M7 code, entered as three planes
    size_t plane_bytes;       // MXFP6+: distance to the second plane of the widened copy, else 0
    unsigned scale_ctas;      // row groups * ceil(nbk/128)
    unsigned widen_ctas;      // CTAs of 256 widening threads (a block or half a block each), 0 when not widened
    // Eq. 4 split of an MXFP4+ operand for the sparse residual MMA (nullptr / 0: not wanted)
    uint8_t* sp_main;         // [rows][K/2]: the nibble plane with BM_H in every BM's place
    uint8_t* sp_res;          // [rows][K/4]: BM_L, 2:1 compressed
    uint8_t* sp_meta;         // [row group of 128][stage of 256 elements][128 rows x 16 bytes]
    int sp_stages;            // ceil(K / 256)
    int sp_row_groups;        // row groups of 128 the metadata covers (two per output tile)
    unsigned split_ctas;      // ceil(row groups * 128 * (nbk / 4) / 256)
};

__device__ __forceinline__ void prepack_scales(const PrepackOperand& op, unsigned id, uint32_t* tile)
{
    const int kgroups = op.nbk >> 2;
    const int kchunks = (kgroups + 31) >> 5;
    const int rg = (int)(id / (unsigned)kchunks), kg0 = (int)(id % (unsigned)kchunks) * 32;
    const int nkg = min(32, kgroups - kg0);
    const uint32_t* src = reinterpret_cast<const uint32_t*>(op.scales);
    for (int i = threadIdx.x; i < 128 * 32; i += 256) {
        const int r = i >> 5, kg = i & 31;
        const int in_tile = (rg & 1) * 128 + r;
        const int64_t row = (int64_t)(rg >> 1) * op.tile_rows + in_tile;
        uint32_t v = 0;
        if (kg < nkg && in_tile < op.tile_rows && row < op.rows) {
            v = src[row * kgroups + kg0 + kg];
            if (op.pp) {
                const uint32_t ix = reinterpret_cast<const uint32_t*>(op.bm_index)[row * kgroups + kg0 + kg];
                uint32_t o = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const uint32_t sb = (v >> (8 * b)) & 255u;
                    o |= (sb - mxpp_shift(sb, (ix >> (8 * b + 5)) & 7u)) << (8 * b);
                }
                v = o;
            }
        }
        tile[kg * 129 + (r & 31) * 4 + (r >> 5)] = v;  // rows of 129 words: no bank conflicts
    }
    __syncthreads();
    uint32_t* dst = reinterpret_cast<uint32_t*>(op.atoms) + ((int64_t)rg * kgroups + kg0) * 128;
    for (int i = threadIdx.x; i < nkg * 128; i += 256) dst[i] = tile[(i >> 7) * 129 + (i & 127)];
}

// Replaces the 6-bit field at bit position `bit` (< 96) of a 16-byte chunk.
__device__ __forceinline__ void set_code6(uint4& v, uint32_t bit, uint32_t code)
{
    const uint32_t wi = bit >> 5, sh = bit & 31u;
    const unsigned long long mask = 63ull << sh, val = (unsigned long long)code << sh;
    uint32_t x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        if (wi == (uint32_t)i) {
            x[i] = (x[i] & ~(uint32_t)mask) | (uint32_t)val;
            x[i + 1] = (x[i + 1] & ~(uint32_t)(mask >> 32)) | (uint32_t)(val >> 32);
        }
    }
    v = make_uint4(x[0], x[1], x[2], x[3]);
}

// MXFP6 / MXFP6+ operand: its sixteen 6-bit codes per half block already are E2M3 codes in the
// bit order the tensor core reads, so they are copied into the 16-byte slot.  The BM of an
// MXFP6+ block, 4 + m/8 with five mantissa bits, is no E2M3 value: it is entered as the sum
// of two that are, 4 + (m >> 2)/2 in the first plane (code s 11 hhh) and (m & 3)/8 in a second
// plane that is zero everywhere else (subnormal code s 00 0ll); the GEMM adds the products of
// both planes (Eq. 4's split at this width, with dense residual passes).
// Sixteen 6-bit codes (x, y, z of `o`) to their 12 bytes: the operand lies packed in global
// memory and the tensor map (16 codes to a 16-byte slot) adds the padding on the way in.
// Threads t (even) and t + 1 are neighbouring lanes and hold the two halves of one block: its 24
// bytes leave as three 8-byte stores, the middle one put together with one shuffle.  All lanes
// of the warp must call it (`live`: this lane has something to store; a block's two halves are
// live or not together).
__device__ __forceinline__ void store_codes6(uint8_t* half0, const uint4 o, bool odd, bool live)
{
    const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, odd ? o.x : o.z, 1);  // even lane: partner's x
    if (!live) return;
    uint2* w = reinterpret_cast<uint2*>(half0);  // the block's first byte: 8-byte aligned
    if (!odd) {
        w[0] = make_uint2(o.x, o.y);
        w[1] = make_uint2(o.z, other);
    } else {
        w[2] = make_uint2(o.y, o.z);
    }
}
__device__ __forceinline__ void widen_six(const PrepackOperand& op, uint32_t t, uint32_t b, bool live)
{
    uint4 o = make_uint4(0u, 0u, 0u, 0u), lo = o;
    if (live) {
        const uint32_t* in = reinterpret_cast<const uint32_t*>(op.nibbles) + (size_t)t * 3u;
        o = make_uint4(in[0], in[1], in[2], 0u);
        const uint32_t sc = op.scales[b];
        if (op.bm_index != nullptr) {
            const uint32_t p = op.bm_index[b] & 31u;
            if ((p >> 4) == (t & 1u)) {
                const uint32_t bit = 6u * (p & 15u);
                const uint32_t x[4] = {o.x, o.y, o.z, o.w};
                const uint32_t wi = bit >> 5;
                const unsigned long long win =
                    (unsigned long long)(wi == 0 ? x[0] : wi == 1 ? x[1] : x[2]) |
                    ((unsigned long long)(wi == 0 ? x[1] : wi == 1 ? x[2] : x[3]) << 32);
                const uint32_t code = (uint32_t)(win >> (bit & 31u)) & 63u;
                const uint32_t sign = code & 32u, m = code & 31u;
                set_code6(o, bit, sign | 0x18u | (m >> 2));
                set_code6(lo, bit, sign | (m & 3u));
            }
        }
        if (sc == 0u) o = lo = make_uint4(0u, 0u, 0u, 0u);
    }
    store_codes6(op.wide + (size_t)b * 24u, o, (t & 1u) != 0u, live);
    if (op.plane_bytes != 0) store_codes6(op.wide + op.plane_bytes + (size_t)b * 24u, lo, (t & 1u) != 0u, live);
}

// One thread per 32 (MXFP4, MXFP4+) or 16 elements (the other modes): 12 or 16 bytes out per 16 codes.
//  * E2M3 (MXFP4 and MXFP4+ operands): the 16 six-bit codes packed into 12 bytes; kind::mxf8f6f4
//    reads 6-bit operands from shared memory as 12 bytes and 4 bytes of padding, which the
//    tensor map's packed 6-bit type adds on the way in, so that global memory and L2 hold 12.
//    The BM of an MX+ block, 4 + m/2 (Eq. 3), is the E2M3 code s 11 mmm.
//  * E4M3 (MX++ operands, whose rescaled values need the exponent range): one byte per code.
// E4M3 code (sign 0) of a positive integer with at most four significant bits.
__device__ __forceinline__ uint32_t e4m3_of_small_int(uint32_t x)
{
    const int msb = 31 - __clz((int)x);
    const uint32_t mant = (msb >= 3 ? x >> (msb - 3) : x << (3 - msb)) & 7u;
    return ((uint32_t)(msb + 7) << 3) | mant;
}

// MXFP8+ (Sec. 4.1 at this width): the BM is stored as sign + seven mantissa bits and means
// 256 + 2 m, which no single E4M3 value holds.  It is entered as the sum of three that do (Eq.
// 4's split, carried one step further): the multiple of 32 below it (at most 448, the largest
// E4M3 value), then the top four significant bits of the rest (at most 62, even) and what is
// left of that (0 or 2).  Plane 0 is the stored plane with the BM replaced, planes 1 and 2 are
// zero except at BM positions; the GEMM's K loop runs once per plane.
__device__ __forceinline__ void widen_eight_plus(const PrepackOperand& op, uint32_t t, uint32_t b)
{
    uint4 o = reinterpret_cast<const uint4*>(op.nibbles)[t];
    uint4 mid = make_uint4(0u, 0u, 0u, 0u), lo = mid;
    const uint32_t sc = op.scales[b];
    const uint32_t p = op.bm_index[b] & 31u;
    if ((p >> 4) == (t & 1u)) {
        const uint32_t e = p & 15u, sh = 8u * (e & 3u);
        uint32_t* ow = e < 4u ? &o.x : e < 8u ? &o.y : e < 12u ? &o.z : &o.w;
        uint32_t* mw = e < 4u ? &mid.x : e < 8u ? &mid.y : e < 12u ? &mid.z : &mid.w;
        uint32_t* lw = e < 4u ? &lo.x : e < 8u ? &lo.y : e < 12u ? &lo.z : &lo.w;
        const uint32_t byte = (*ow >> sh) & 255u;
        const uint32_t sign = byte & 0x80u, v = 256u + 2u * (byte & 0x7Fu);
        const uint32_t hi = min(v & ~31u, 448u), rem = v - hi;
        *ow = (*ow & ~(255u << sh)) | ((sign | 0x78u | ((hi - 256u) >> 5)) << sh);
        if (rem != 0u) {
            const int msb = 31 - __clz((int)rem);
            const uint32_t keep = msb > 3 ? (rem >> (msb - 3)) << (msb - 3) : rem;
            *mw = (sign | e4m3_of_small_int(keep)) << sh;
            if (rem != keep) *lw = (sign | e4m3_of_small_int(rem - keep)) << sh;
        }
    }
    if (sc == 0u) o = mid = lo = make_uint4(0u, 0u, 0u, 0u);
    uint8_t* dst = op.wide + (size_t)t * 16u;
    *reinterpret_cast<uint4*>(dst) = o;
    *reinterpret_cast<uint4*>(dst + op.plane_bytes) = mid;
    *reinterpret_cast<uint4*>(dst + 2 * op.plane_bytes) = lo;
}

__device__ __forceinline__ void widen_codes(const PrepackOperand& op, unsigned id)
{
    if (!op.pp && !op.eight_plus && !op.eight && !op.six) {
        // MXFP4 / MXFP4+ -> E2M3: a thread per block, 16 bytes in, 24 bytes out
        const uint32_t blk = id * 256u + threadIdx.x;
        if (blk >= (uint32_t)op.rows * (uint32_t)op.nbk) return;
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(op.nibbles) + blk);
        const uint32_t p = op.bm_index != nullptr ? op.bm_index[blk] & 31u : 32u;
        // Eq. 3, BM branch included, in the half that holds the BM
        uint4 s0 = e2m1x16_to_e2m3_slot(w.x, w.y, p < 16u ? p : 16u);
        uint4 s1 = e2m1x16_to_e2m3_slot(w.z, w.w, (p >= 16u && p < 32u) ? p - 16u : 16u);
        if (op.scales[blk] == 0u) s0 = s1 = make_uint4(0u, 0u, 0u, 0u);
        uint2* out = reinterpret_cast<uint2*>(op.wide + (size_t)blk * 24u);
        out[0] = make_uint2(s0.x, s0.y);
        out[1] = make_uint2(s0.z, s1.x);
        out[2] = make_uint2(s1.y, s1.z);
        return;
    }
    const uint32_t t = id * 256u + threadIdx.x;  // half block: 16 elements
    const uint32_t b = t >> 1;
    const bool live = b < (uint32_t)op.rows * (uint32_t)op.nbk;
    if (op.six) return widen_six(op, t, b, live);  // (every lane takes part in its stores)
    if (!live) return;
    if (op.eight_plus) return widen_eight_plus(op, t, b);
    if (op.eight) {
        // MXFP8: one byte per element already; a flushed block's codes are zero by construction
        reinterpret_cast<uint4*>(op.wide)[t] = reinterpret_cast<const uint4*>(op.nibbles)[t];
        return;
    }
    const uint2 w = reinterpret_cast<const uint2*>(op.nibbles)[t];
    const uint32_t sc = op.scales[b];
    const uint32_t ib = op.bm_index != nullptr ? op.bm_index[b] : 0u;
    // the BM, if this half block holds it: element e, code nib
    const uint32_t p = ib & 31u;
    const uint32_t e = p & 15u;
    const uint32_t nib = (((e & 8u) ? w.y : w.x) >> ((e & 7u) * 4u)) & 15u;
    const bool has_bm = op.bm_index != nullptr && (p >> 4) == (t & 1u);
    uint8_t* dst = op.wide + (size_t)t * 16u;
    // MX++: BM scaled up by 2^shift, NBMs down by 2^-(delta - shift) (see mxpp_shift)
    const uint32_t delta = ib >> 5;
    const uint32_t shift = mxpp_shift(sc, delta);
    const uint2 lut = kE4m3Lut[delta - shift];
    uint4 o;
    o.x = e2m1x4_to_e4m3x4(w.x, lut);
    o.y = e2m1x4_to_e4m3x4(w.x >> 16, lut);
    o.z = e2m1x4_to_e4m3x4(w.y, lut);
    o.w = e2m1x4_to_e4m3x4(w.y >> 16, lut);
    if (sc == 0u) o = make_uint4(0u, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(dst) = o;
    // Eq. 3, BM branch.  Same thread, later store to the same bytes: lands after the vector
    // store above.
    if (has_bm && sc != 0u)
        dst[e] = (uint8_t)(((nib & 8u) << 4) | (0x48u + (shift << 3)) | (nib & 7u));
}

// Eq. 4 / Algorithm 1 (ReplaceBM, MakeFragment) done once per operand instead of once per tile:
// one thread per 128 elements of a row (four blocks: one K group of the sparse instruction).
//   main plane: the block's codes with the BM's code s m2 m1 m0 replaced by BM_H = s 1 1 m2
//     (4 or 6);
//   residual: BM_L = s 0 m1 m0 (0, 0.5, 1, 1.5) as the only non-zero of the block, compressed
//     2:1 the way tcgen05.mma.sp reads it: of each 8 consecutive elements two aligned pairs are
//     kept (4 codes), and a nibble of metadata names the pairs -- low two bits the first, high
//     two bits the second, ascending.  The group of 8 that holds the BM keeps the BM's pair and
//     pair 3 (pairs 0 and 3 if the BM sits in pair 3); every other group keeps pairs 0 and 1.
//   Blocks with scale byte 0 become zeros in both.  Rows past the operand's end (the row groups
//   are whole) get metadata only, so that every nibble the tensor core reads is a valid one.
__device__ __forceinline__ void split_codes(const PrepackOperand& op, unsigned id)
{
    const uint32_t t = id * 256u + threadIdx.x;
    const uint32_t kgroups = (uint32_t)op.nbk >> 2;
    if (t >= (uint32_t)op.sp_row_groups * 128u * kgroups) return;
    const uint32_t row = t / kgroups, g = t - row * kgroups;
    uint8_t* meta_dst = op.sp_meta + ((size_t)(row >> 7) * (size_t)op.sp_stages + (g >> 1)) * 2048u +
                        (row & 127u) * 16u + (g & 1u) * 8u;
    unsigned long long meta = 0x4444444444444444ull;
    if (row < (uint32_t)op.rows) {
        const size_t b0 = (size_t)row * (size_t)op.nbk + 4u * g;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const uint4 c = __ldg(reinterpret_cast<const uint4*>(op.nibbles) + b0 + b);
            uint32_t w[4] = {c.x, c.y, c.z, c.w};
            const uint32_t sc = op.scales[b0 + b];
            unsigned long long res = 0ull;
            if (sc == 0u) {
                w[0] = w[1] = w[2] = w[3] = 0u;
            } else {
                const uint32_t pos = op.bm_index[b0 + b] & 31u;
                const uint32_t sh = (pos & 7u) * 4u;
                uint32_t word = pos < 8u ? w[0] : pos < 16u ? w[1] : pos < 24u ? w[2] : w[3];
                const uint32_t nib = (word >> sh) & 15u;
                word = (word & ~(15u << sh)) | (((nib & 8u) | 6u | ((nib >> 2) & 1u)) << sh);
                if (pos < 8u) w[0] = word; else if (pos < 16u) w[1] = word; else if (pos < 24u) w[2] = word; else w[3] = word;
                const uint32_t gi = pos >> 3, pair = (pos & 7u) >> 1, slot = pair == 3u ? 1u : 0u;
                const uint32_t mnib = pair == 3u ? 0xCu : (pair | 0xCu);
                meta = (meta & ~(15ull << (16 * b + 4 * gi))) | ((unsigned long long)mnib << (16 * b + 4 * gi));
                if (nib & 3u)
                    res = (unsigned long long)((nib & 8u) | (nib & 3u)) << (4u * (4u * gi + 2u * slot + (pos & 1u)));
            }
            reinterpret_cast<uint4*>(op.sp_main)[b0 + b] = make_uint4(w[0], w[1], w[2], w[3]);
            reinterpret_cast<unsigned long long*>(op.sp_res)[b0 + b] = res;
        }
    }
    *reinterpret_cast<unsigned long long*>(meta_dst) = meta;
    // an odd number of K groups: the last stage's second group does not exist, its metadata must
    if (g == kgroups - 1u && (kgroups & 1u))
        *reinterpret_cast<unsigned long long*>(meta_dst + 8) = 0x4444444444444444ull;
}

__global__ void __launch_bounds__(256) prepack_kernel(const PrepackOperand a, const PrepackOperand b,
                                                      StatusBlock* status)
{
    __shared__ uint32_t tile[32 * 129];
    unsigned id = blockIdx.x;
    if (id == 0 && threadIdx.x == 0 && status != nullptr) {
        status->code = 0u;  // the GEMM that follows on the stream reports into this block
        status->where = 0u;
        __threadfence();
    }
    // the GEMM's prologue may start while this grid drains (its first CTA has cleared the status
    // block by then: a dependent grid is released only when every CTA has passed this point)
    ptx::grid_launch_dependents();
    if (id < a.scale_ctas) return prepack_scales(a, id, tile);
    id -= a.scale_ctas;
    if (id < b.scale_ctas) return prepack_scales(b, id, tile);
    id -= b.scale_ctas;
    if (id < a.widen_ctas) return widen_codes(a, id);
    id -= a.widen_ctas;
    if (id < b.widen_ctas) return widen_codes(b, id);
    id -= b.widen_ctas;
    if (id < a.split_ctas) return split_codes(a, id);
    id -= a.split_ctas;
    split_codes(b, id);
}

#ifndef MXP_S_L2PROMO
#define MXP_S_L2PROMO CU_TENSOR_MAP_L2_PROMOTION_L2_256B
#endif
// 2-D byte tensor [rows][row_bytes], boxes of 128 bytes x box_rows rows, 128B swizzle.
bool make_tmap_rows(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t row_bytes, int box_rows)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)kRowBytes, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              MXP_S_L2PROMO, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D tensor of 6-bit codes [rows][K], 16 codes packed into 12 bytes in global memory and spread
// into 16-byte slots in shared memory (the form kind::mxf8f6f4 reads): boxes of 128 codes (a
// 128-byte swizzle span in shared memory) x box_rows rows.  The base must be 32-byte aligned and
// K a multiple of 128; the innermost coordinate of a copy is in codes, a multiple of 128.
bool make_tmap_rows6(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t K, int box_rows)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 3 / 4};
    const cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_16U6_ALIGN16B, 2, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              MXP_S_L2PROMO, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Scale atoms as a 3-D tensor of 32-bit words [row groups][K groups][128], boxes of
// 128 x kgroups_per_stage x rgs.
bool make_tmap_atoms(CUtensorMap* m, const uint8_t* base, int64_t rgs_total, int64_t kgroups,
                     int box_kg, int box_rg)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {128u, (cuuint64_t)kgroups, (cuuint64_t)rgs_total};
    const cuuint64_t strides[2] = {(cuuint64_t)kAtom, (cuuint64_t)kAtom * (cuuint64_t)kgroups};
    const cuuint32_t box[3] = {128u, (cuuint32_t)box_kg, (cuuint32_t)box_rg};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Layout {
    size_t sfa, sfb, wa, wb, total;
};

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// scale row groups (atoms of 128 rows) of an operand whose output tiles take `tile_rows` rows
inline int64_t row_groups(int64_t rows, int tile_rows) { return 2 * ((rows + tile_rows - 1) / tile_rows); }

// E2M3 planes an operand is widened into: two for MXFP6+ (see widen_six), else one.
inline int mode_parts(mxp_mode m)
{
    return m == MXP_MODE_MXFP6_PLUS ? 2 : m == MXP_MODE_MXFP8_PLUS ? 3 : 1;
}
inline bool mode_six(mxp_mode m) { return m == MXP_MODE_MXFP6 || m == MXP_MODE_MXFP6_PLUS; }
inline bool mode_eight(mxp_mode m) { return m == MXP_MODE_MXFP8 || m == MXP_MODE_MXFP8_PLUS; }
// Bits per code of an operand's widened form: E4M3 bytes for MX++ and MXFP8(+), E2M3 codes
// packed 16 to 12 bytes for the rest.
inline int wide_bits(mxp_mode m) { return (m == MXP_MODE_MXFP4_PP || mode_eight(m)) ? 8 : 6; }
inline bool mode_plus(mxp_mode m)
{
    return m == MXP_MODE_MXFP4_PLUS || m == MXP_MODE_MXFP4_PP || m == MXP_MODE_MXFP6_PLUS ||
           m == MXP_MODE_MXFP8_PLUS;
}

// Sized for either tiling of B's scales (the tile shape is chosen per call).
Layout layout(int64_t M, int64_t N, int64_t K, bool wide, int parts_a = 1, int parts_b = 1)
{
    Layout l;
    const size_t kgroups = (size_t)(K / 128);
    size_t off = kStatusBytes;
    off = round_up(off, 1024);
    l.sfa = off;
    off += (size_t)row_groups(M, kTileM) * kgroups * kAtom;
    off = round_up(off, 1024);
    l.sfb = off;
    off += (size_t)std::max(row_groups(N, sub_n(wide, 1)), row_groups(N, sub_n(wide, 2))) * kgroups * kAtom;
    off = round_up(off, 1024);
    l.wa = off;
    if (wide) off += (size_t)M * (size_t)K * (size_t)parts_a;
    off = round_up(off, 1024);
    l.wb = off;
    if (wide) off += (size_t)N * (size_t)K * (size_t)parts_b;
    l.total = round_up(off, 1024);
    return l;
}

// Two halves per tile unless that leaves the last wave of tiles much emptier than single
// halves would: compare the columns each CTA pair walks through either way.
int choose_halves(int64_t M, int64_t N, bool wide, int num_sms)
{
    const int forced = override_get(MXP_KNOB_STREAM_HALVES);  // tests and measurements
    if (forced == 1 || forced == 2) return forced;
    const int64_t clusters = num_sms / 2, tiles_m = (M + kTileM - 1) / kTileM;
    auto cost = [&](int h) {  // columns a CTA pair walks through
        const int64_t tile_n = (int64_t)h * sub_n(wide, h);
        const int64_t tiles = tiles_m * ((N + tile_n - 1) / tile_n);
        return (tiles + clusters - 1) / clusters * tile_n;
    };
    return cost(1) < cost(2) ? 1 : 2;
}

template <bool kWide, int kHalves, bool kSparse, typename OutT>
mxp_status launch_stream(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tsa,
                         const CUtensorMap& tsb, const CUtensorMap& tres, const CUtensorMap& tmeta,
                         const SParams& prm, int num_sms, cudaStream_t stream)
{
    using C = SCfg<kWide, kHalves, kSparse>;
    auto kern = gemm_tc_stream_kernel<kWide, kHalves, kSparse, OutT>;
    static SmemAttrOnce once;
    if (ensure_dynamic_smem(kern, C::kSmem, once) != cudaSuccess) return MXP_ERR_CUDA;
    const int64_t tiles =
        (int64_t)((prm.M + kTileM - 1) / kTileM) * ((prm.N + C::kTileN - 1) / C::kTileN);
    int64_t clusters = num_sms / 2;
    if (tiles < clusters) clusters = tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, ta, tb, tsa, tsb, tres, tmeta, prm) == cudaSuccess ? MXP_OK
                                                                                             : MXP_ERR_CUDA;
}

// Weight-only form at prefill sizes (Sec. 7.1, "conversion before computation"; the paper's
// matmul table runs M up to 4096): dense bf16 activations become an operand of the same
// tensor-core kernel.  A bf16 value has eight significant bits, an E4M3 value four, so x = hi +
// lo with hi = x cut to four significant bits and lo the rest, both scaled by the block's power
// of two 2^(floor(log2 amax) - 7) (largest scaled magnitude below 256, inside E4M3's 448).  hi
// is always exact; lo is exact for elements within 2^9 of the block's maximum and otherwise
// rounded at 2^-10 in scaled units, i.e. below 2^-17 of the block maximum.  Two planes with
// one E8M0 scale per block of 32: the K loop runs once per plane, like an MXFP6+ operand.
// One thread per block of 32; rows past M (up to the next multiple of 128) get scale byte 0.
__global__ void __launch_bounds__(256)
prepack_dense_kernel(const __nv_bfloat16* __restrict__ A, int64_t lda, int M, int rows_pad, int nbk,
                     uint8_t* __restrict__ atoms, uint4* __restrict__ slots, size_t plane_slots,
                     StatusBlock* status)
{
    const int64_t blk = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (blk == 0 && status != nullptr) {
        status->code = 0u;
        status->where = 0u;
        __threadfence();
    }
    ptx::grid_launch_dependents();  // the GEMM's prologue may start while this grid drains
    const int64_t row = blk / nbk;
    const int kb = (int)(blk - row * nbk);
    if (row >= rows_pad) return;
    uint32_t sb = 0;
    if (row < M) {
        const uint4* src = reinterpret_cast<const uint4*>(A + row * lda + (int64_t)kb * 32);
        uint32_t x[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 v = __ldg(src + i);
            x[4 * i] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
        }
        uint32_t mx = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) mx = max(mx, max(x[i] & 0x7FFFu, (x[i] >> 16) & 0x7FFFu));
        const uint32_t E = mx >> 7;  // exponent field of the block's largest magnitude
        sb = E > 7u ? E - 7u : 0u;
        const float inv = __uint_as_float((254u - sb) << 23);  // 2^(127 - sb)
        uint32_t hi[8], lo[8];  // four E4M3 codes per word
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t h = 0, l = 0;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t w = x[2 * i + j];
                const float x0 = __uint_as_float(w << 16), x1 = __uint_as_float(w & 0xFFFF0000u);
                const float h0 = __uint_as_float((w << 16) & 0xFFF00000u);
                const float h1 = __uint_as_float(w & 0xFFF00000u);
                uint16_t hc, lc;
                asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hc) : "f"(h1 * inv), "f"(h0 * inv));
                asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;"
                    : "=h"(lc)
                    : "f"((x1 - h1) * inv), "f"((x0 - h0) * inv));
                h |= (uint32_t)hc << (16 * j);
                l |= (uint32_t)lc << (16 * j);
            }
            hi[i] = h;
            lo[i] = l;
        }
        uint4* dst = slots + (row * nbk + kb) * 2;
        dst[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        dst[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        dst[plane_slots] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        dst[plane_slots + 1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
    }
    const int r = (int)(row & 127);
    atoms[((row >> 7) * (nbk >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (kb & 3)] = (uint8_t)sb;
}

}  // namespace

size_t stream_dense_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode b_mode)
{
    if (M < 1 || N < 1 || K % 128 != 0 || b_mode > MXP_MODE_MXFP8_PLUS) return 0;
    if ((uint64_t)M * (uint64_t)K / 16 >= (1ull << 31) || (uint64_t)N * (uint64_t)K / 16 >= (1ull << 32))
        return 0;
    return layout(M, N, K, true, 2, mode_parts(b_mode)).total;
}

size_t stream_dense_prepacked_workspace_bytes(int64_t M, int64_t K)
{
    if (M < 1 || K < 128 || K % 128 != 0 || (uint64_t)M * (uint64_t)K / 16 >= (1ull << 31)) return 0;
    return layout(M, 0, K, true, 2, 1).total;
}

size_t stream_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode a_mode, mxp_mode b_mode)
{
    // Small M or N is better served by the in-place single-CTA kernel, except for MX++
    // operands, which only this path handles (rows past the end are zero-filled by TMA).
    // (and MXFP6 operands, likewise)
    const bool pp = a_mode == MXP_MODE_MXFP4_PP || b_mode == MXP_MODE_MXFP4_PP ||
                    mode_six(a_mode) || mode_six(b_mode) || mode_eight(a_mode) || mode_eight(b_mode);
    if (M < 1 || N < 1 || K % 128 != 0) return 0;
    if (!pp && (M <= 128 || N <= 128)) return 0;
    // the prepack kernel indexes half blocks (16 elements) of an operand with 32 bits
    if ((uint64_t)M * (uint64_t)K / 16 >= (1ull << 32) || (uint64_t)N * (uint64_t)K / 16 >= (1ull << 32))
        return 0;
    const bool wide = a_mode != MXP_MODE_MXFP4 || b_mode != MXP_MODE_MXFP4;
    if (a_mode > MXP_MODE_MXFP8_PLUS || b_mode > MXP_MODE_MXFP8_PLUS) return 0;
    return layout(M, N, K, wide, mode_parts(a_mode), mode_parts(b_mode)).total;
}

namespace {
// Prepacked form of the B operand in a caller-owned buffer: scale atoms, then (wide) the
// widened codes.
struct PackedLayout {
    size_t atoms[2];  // scale atoms tiled for one-half tiles, for two-half tiles
    size_t wide, total;
};
// bits: 0 (scale atoms only), 6 or 8 (widened codes behind them, `parts` planes of them)
PackedLayout packed_layout(int64_t rows, int64_t K, int bits, int parts = 1)
{
    const bool wide = bits != 0;
    PackedLayout l;
    l.atoms[0] = 0;
    l.atoms[1] = round_up((size_t)row_groups(rows, sub_n(wide, 1)) * (size_t)(K / 128) * kAtom, 1024);
    l.wide = l.atoms[1] +
             round_up((size_t)row_groups(rows, sub_n(wide, 2)) * (size_t)(K / 128) * kAtom, 1024);
    l.total = l.wide + round_up((size_t)parts * (size_t)rows * (size_t)K * (size_t)bits / 8, 1024);
    return l;
}

PrepackOperand prepack_operand(const mxp_packed& P, int64_t rows, int64_t K, bool wide, int tile_rows,
                               uint8_t* atoms, uint8_t* wide_bytes)
{
    const int nbk = (int)(K / 32);
    const int kgroups = nbk / 4;
    PrepackOperand op;
    op.nibbles = P.nibbles;
    op.scales = P.scales;
    op.bm_index = mode_plus(P.mode) ? P.bm_index : nullptr;
    op.pp = P.mode == MXP_MODE_MXFP4_PP;
    op.six = mode_six(P.mode);
    op.eight = P.mode == MXP_MODE_MXFP8;
    op.eight_plus = P.mode == MXP_MODE_MXFP8_PLUS;
    op.plane_bytes = mode_parts(P.mode) > 1 ? (size_t)rows * (size_t)K * (size_t)wide_bits(P.mode) / 8 : 0;
    op.atoms = atoms;
    op.wide = wide ? wide_bytes : nullptr;
    op.rows = (int)rows;
    op.nbk = nbk;
    op.tile_rows = tile_rows;
    op.scale_ctas = (unsigned)(row_groups(rows, tile_rows) * ((kgroups + 31) / 32));
    // a thread per block for the 4-bit modes that widen to E2M3, per half block otherwise
    const bool per_block = !op.pp && !op.six && !op.eight && !op.eight_plus;
    op.widen_ctas = wide ? (unsigned)((rows * nbk * (per_block ? 1 : 2) + 255) / 256) : 0u;
    op.sp_main = op.sp_res = op.sp_meta = nullptr;
    op.sp_stages = op.sp_row_groups = 0;
    op.split_ctas = 0u;
    return op;
}

// Prepacked form of an MXFP4+ operand that takes the A slot of the sparse-residual kernel: scale
// atoms tiled for 256-row output tiles, then the three planes split_codes() writes.
struct SplitLayout {
    size_t atoms, main, res, meta, total;
};
SplitLayout split_layout(int64_t rows, int64_t K)
{
    SplitLayout l;
    const size_t rgs = (size_t)row_groups(rows, kTileM), kgroups = (size_t)(K / 128);
    l.atoms = 0;
    l.main = round_up(rgs * kgroups * kAtom, 1024);
    l.res = l.main + round_up((size_t)rows * (size_t)K / 2, 1024);
    l.meta = l.res + round_up((size_t)rows * (size_t)K / 4, 1024);
    l.total = l.meta + round_up(rgs * (size_t)((K + 255) / 256) * 2048, 1024);
    return l;
}
PrepackOperand split_operand(const mxp_packed& P, uint8_t* base)
{
    const SplitLayout l = split_layout(P.rows, P.cols);
    PrepackOperand op = prepack_operand(P, P.rows, P.cols, false, kTileM, base + l.atoms, nullptr);
    op.sp_main = base + l.main;
    op.sp_res = base + l.res;
    op.sp_meta = base + l.meta;
    op.sp_stages = (int)((P.cols + 255) / 256);
    op.sp_row_groups = (int)row_groups(P.rows, kTileM);
    op.split_ctas = (unsigned)(((int64_t)op.sp_row_groups * 128 * (P.cols / 128) + 255) / 256);
    return op;
}
// 2-D byte tensor [rows][row_bytes], boxes of 64 bytes x 128 rows, 64-byte swizzle (the
// compressed residual tile of the sparse instruction).
bool make_tmap_rows64(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t row_bytes)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {64u, 128u};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
              MXP_S_L2PROMO, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Sparsity metadata [row groups][stages][2048 bytes] as 32-bit words, one box = one stage's
// 128 rows x 16 bytes.
bool make_tmap_meta(CUtensorMap* m, const uint8_t* base, int64_t row_groups_total, int64_t stages)
{
    EncodeFn fn = tensormap_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {128u, (cuuint64_t)(4 * stages), (cuuint64_t)row_groups_total};
    const cuuint64_t strides[2] = {512u, (cuuint64_t)2048 * (cuuint64_t)stages};
    const cuuint32_t box[3] = {128u, 4u, 1u};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Workspace of a sparse-residual call: status block, then what is not prepacked -- the MX+
// operand's split form, the plain operand's scale atoms (sized for either tiling).
struct SparseLayout {
    size_t x, y, total;
};
SparseLayout sparse_layout(int64_t rows_x, int64_t rows_y, int64_t K, bool x_prepacked, bool y_prepacked)
{
    SparseLayout l;
    size_t off = round_up(kStatusBytes, 1024);
    l.x = off;
    if (!x_prepacked) off += split_layout(rows_x, K).total;
    l.y = off;
    if (!y_prepacked)
        off += round_up((size_t)std::max(row_groups(rows_y, sub_n(false, 1)), row_groups(rows_y, sub_n(false, 2))) *
                            (size_t)(K / 128) * kAtom, 1024);
    l.total = off;
    return l;
}
PrepackOperand no_operand()
{
    PrepackOperand op = {};
    return op;
}
}  // namespace

size_t stream_prepack_bytes(int64_t rows, int64_t K, int form)
{
    if (rows <= 0 || K <= 0 || K % 128 != 0 || form < 0 || form > MXP_PREPACK_WIDE8_X3) return 0;
    if ((uint64_t)rows * (uint64_t)K / 16 >= (1ull << 32)) return 0;
    if (form == MXP_PREPACK_SPLIT) return split_layout(rows, K).total;
    if (form == MXP_PREPACK_WIDE_X2) return packed_layout(rows, K, 6, 2).total;
    if (form == MXP_PREPACK_WIDE8_X3) return packed_layout(rows, K, 8, 3).total;
    return packed_layout(rows, K, form == MXP_PREPACK_WIDE ? 6 : form == MXP_PREPACK_WIDE8 ? 8 : 0).total;
}

int stream_wide_form(mxp_mode b_mode)
{
    if (b_mode == MXP_MODE_MXFP6_PLUS) return MXP_PREPACK_WIDE_X2;   // its BM is the sum of two E2M3 planes
    if (b_mode == MXP_MODE_MXFP8_PLUS) return MXP_PREPACK_WIDE8_X3;  // ... of three E4M3 planes
    return wide_bits(b_mode) == 8 ? MXP_PREPACK_WIDE8 : MXP_PREPACK_WIDE;
}

mxp_status stream_prepack(const mxp_packed& P, int form, void* out, size_t out_bytes,
                          cudaStream_t stream)
{
    const bool wide = form != MXP_PREPACK_PLAIN && form != MXP_PREPACK_SPLIT;
    const size_t need = stream_prepack_bytes(P.rows, P.cols, form);
    if (need == 0) return MXP_ERR_UNSUPPORTED;
    if (wide && form != stream_wide_form(P.mode)) return MXP_ERR_INVALID_ARG;  // 6-bit codes or bytes: the mode's
    if (form == MXP_PREPACK_SPLIT) {
        if (P.mode != MXP_MODE_MXFP4_PLUS) return MXP_ERR_UNSUPPORTED;
        if (out == nullptr || out_bytes < need) return MXP_ERR_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(out) & 255) || (reinterpret_cast<uintptr_t>(P.nibbles) & 15) ||
            (reinterpret_cast<uintptr_t>(P.scales) & 3))
            return MXP_ERR_INVALID_ARG;
        const PrepackOperand px = split_operand(P, static_cast<uint8_t*>(out));
        const uint64_t ctas = (uint64_t)px.scale_ctas + px.split_ctas;
        if (ctas > 0x7FFFFFFFull) return MXP_ERR_UNSUPPORTED;
        prepack_kernel<<<(unsigned)ctas, 256, 0, stream>>>(px, no_operand(), nullptr);
        return cudaGetLastError() == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
    }
    if ((mode_six(P.mode) || mode_eight(P.mode)) && !wide) return MXP_ERR_UNSUPPORTED;
    if (out == nullptr || out_bytes < need) return MXP_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(out) & 255) || (reinterpret_cast<uintptr_t>(P.nibbles) & 15) ||
        (reinterpret_cast<uintptr_t>(P.scales) & 3) ||
        (P.mode == MXP_MODE_MXFP4_PP && (reinterpret_cast<uintptr_t>(P.bm_index) & 3)))
        return MXP_ERR_INVALID_ARG;
    const PackedLayout l = packed_layout(P.rows, P.cols, wide ? wide_bits(P.mode) : 0, mode_parts(P.mode));
    uint8_t* o = static_cast<uint8_t*>(out);
    // both tilings of the scales (the GEMM picks its tile shape per call); widened bytes once
    const PrepackOperand p1 =
        prepack_operand(P, P.rows, P.cols, wide, sub_n(wide, 1), o + l.atoms[0], o + l.wide);
    PrepackOperand p2 =
        prepack_operand(P, P.rows, P.cols, wide, sub_n(wide, 2), o + l.atoms[1], o + l.wide);
    p2.widen_ctas = 0;
    const uint64_t ctas = (uint64_t)p1.scale_ctas + p2.scale_ctas + p1.widen_ctas;
    if (ctas > 0x7FFFFFFFull) return MXP_ERR_UNSUPPORTED;
    prepack_kernel<<<(unsigned)ctas, 256, 0, stream>>>(p1, p2, nullptr);
    return cudaGetLastError() == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

// Where a quantizer that prepares A for the GEMM itself has to write inside the workspace of a
// call with a prepacked B (mxp_quantize_gemm_ready): scale atoms and 16-byte code slots.
bool stream_a_ready_layout(int64_t M, int64_t K, size_t* atoms, size_t* slots, size_t* total)
{
    if (M <= 128 || K <= 0 || K % 128 != 0 || (uint64_t)M * (uint64_t)K / 16 >= (1ull << 32)) return false;
    const Layout l = layout(M, 0, K, true);
    *atoms = l.sfa;
    *slots = l.wa;
    *total = l.total;
    return true;
}

// `b_prepacked` (may be nullptr): B already in the form stream_prepack() writes for the same
// `wide`; then only A is prepared here and the workspace needs no room for B.
mxp_status launch_gemm_tc_stream(int64_t M, int64_t N, int64_t K, const mxp_packed& A,
                                 const mxp_packed& B, const void* b_prepacked, void* D,
                                 mxp_dtype d_dt, int64_t ldd, void* workspace,
                                 size_t workspace_bytes, cudaStream_t stream, bool a_ready,
                                 const void* a_dense, int64_t lda)
{
    // `a_dense`: bf16 activations (weight-only form); `A` is then a placeholder of mode MXFP4
    const bool dense = a_dense != nullptr;
    if (dense && a_ready) return MXP_ERR_UNSUPPORTED;
    const bool ap = A.mode != MXP_MODE_MXFP4, bp = B.mode != MXP_MODE_MXFP4;
    const bool wide = ap || bp || a_ready || dense;
    // `a_ready`: A's atoms and code slots are in the workspace already (and the status block is
    // cleared); needs a prepacked B, so that nothing is left to prepare
    if (a_ready && (b_prepacked == nullptr || A.mode > MXP_MODE_MXFP4_PLUS)) return MXP_ERR_UNSUPPORTED;
    if (A.mode > MXP_MODE_MXFP8_PLUS || B.mode > MXP_MODE_MXFP8_PLUS) return MXP_ERR_UNSUPPORTED;
    const int parts_a = dense ? 2 : mode_parts(A.mode), parts_b = mode_parts(B.mode);
    const Layout l = layout(M, b_prepacked ? 0 : N, K, wide, parts_a, parts_b);
    if (workspace == nullptr || workspace_bytes < l.total) return MXP_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return MXP_ERR_INVALID_ARG;
    if (b_prepacked != nullptr && (reinterpret_cast<uintptr_t>(b_prepacked) & 255))
        return MXP_ERR_INVALID_ARG;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int num_sms = sm_count();
    if (num_sms <= 0) return MXP_ERR_CUDA;
    const int nbk = (int)(K / 32);
    const int kgroups = nbk / 4;
    const int halves = choose_halves(M, N, wide, num_sms);
    const int sub = sub_n(wide, halves);
    const int rga = (int)row_groups(M, kTileM), rgb = (int)row_groups(N, sub);
    if (((dense ? reinterpret_cast<uintptr_t>(a_dense) : reinterpret_cast<uintptr_t>(A.nibbles)) |
         reinterpret_cast<uintptr_t>(B.nibbles)) & 15)
        return MXP_ERR_INVALID_ARG;
    if (dense && (lda < K || lda % 8 != 0)) return MXP_ERR_INVALID_ARG;
    // the widening threads index their operand with 32 bits
    if ((uint64_t)M * nbk * 2 >= (1ull << 32) || (uint64_t)N * nbk * 2 >= (1ull << 32))
        return MXP_ERR_UNSUPPORTED;
    // MX++: the scale re-tiling reads the index plane a word at a time
    if ((A.mode == MXP_MODE_MXFP4_PP && (reinterpret_cast<uintptr_t>(A.bm_index) & 3)) ||
        (B.mode == MXP_MODE_MXFP4_PP && (reinterpret_cast<uintptr_t>(B.bm_index) & 3)))
        return MXP_ERR_INVALID_ARG;

    const PackedLayout lb = packed_layout(N, K, wide ? wide_bits(B.mode) : 0, parts_b);
    const uint8_t* b_atoms =
        b_prepacked ? static_cast<const uint8_t*>(b_prepacked) + lb.atoms[halves - 1] : ws + l.sfb;
    const uint8_t* b_wide = b_prepacked ? static_cast<const uint8_t*>(b_prepacked) + lb.wide : ws + l.wb;
    if (dense) {
        const int rows_pad = rga * 128;
        const int64_t blocks = (int64_t)rows_pad * nbk;
        prepack_dense_kernel<<<(unsigned)((blocks + 255) / 256), 256, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(a_dense), lda, (int)M, rows_pad, nbk, ws + l.sfa,
            reinterpret_cast<uint4*>(ws + l.wa), (size_t)M * (size_t)K / 16,
            static_cast<StatusBlock*>(workspace));
        if (cudaGetLastError() != cudaSuccess) return MXP_ERR_CUDA;
    }
    const PrepackOperand pa = (a_ready || dense)
                                  ? no_operand()
                                  : prepack_operand(A, M, K, wide, kTileM, ws + l.sfa, ws + l.wa);
    const PrepackOperand pb =
        b_prepacked ? no_operand() : prepack_operand(B, N, K, wide, sub, ws + l.sfb, ws + l.wb);
    const uint64_t ctas = (uint64_t)pa.scale_ctas + pb.scale_ctas + pa.widen_ctas + pb.widen_ctas;
    if (ctas > 0x7FFFFFFFull) return MXP_ERR_UNSUPPORTED;
    if (ctas != 0) {
        prepack_kernel<<<(unsigned)ctas, 256, 0, stream>>>(pa, pb, static_cast<StatusBlock*>(workspace));
        if (cudaGetLastError() != cudaSuccess) return MXP_ERR_CUDA;
    }

    CUtensorMap ta, tb, tsa, tsb;
    const int box_kg = wide ? 1 : 2;
    const bool maps_ok =
        (wide ? ((dense || wide_bits(A.mode) == 8) ? make_tmap_rows(&ta, ws + l.wa, M * parts_a, K, 128)
                                                     : make_tmap_rows6(&ta, ws + l.wa, M * parts_a, K, 128)) &&
                    (wide_bits(B.mode) == 8 ? make_tmap_rows(&tb, b_wide, N * parts_b, K, sub / 2)
                                            : make_tmap_rows6(&tb, b_wide, N * parts_b, K, sub / 2))
              : make_tmap_rows(&ta, A.nibbles, M, K / 2, 128) &&
                    make_tmap_rows(&tb, B.nibbles, N, K / 2, sub / 2)) &&
        make_tmap_atoms(&tsa, ws + l.sfa, rga, kgroups, box_kg, 1) &&
        make_tmap_atoms(&tsb, b_atoms, rgb, kgroups, box_kg, 2 * halves);
    if (!maps_ok) return MXP_ERR_CUDA;

    SParams prm;
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.a_fmt = (dense || A.mode == MXP_MODE_MXFP4_PP || mode_eight(A.mode)) ? kFmtE4M3 : kFmtE2M3;
    prm.b_fmt = (B.mode == MXP_MODE_MXFP4_PP || mode_eight(B.mode)) ? kFmtE4M3 : kFmtE2M3;
    prm.parts_a = parts_a;
    prm.parts_b = parts_b;
    prm.D = D;
    prm.ldd = ldd;
    prm.d_vec_ok = ((reinterpret_cast<uintptr_t>(D) & 15) == 0) &&
                   ((ldd * (d_dt == MXP_BF16 ? 2 : 4)) % 16 == 0);
    prm.transposed = 0;
    prm.status = static_cast<StatusBlock*>(workspace);
    const bool f32 = d_dt == MXP_F32;
#define MXP_S_LAUNCH(W, H)                                                                    \
    (f32 ? launch_stream<W, H, false, float>(ta, tb, tsa, tsb, ta, ta, prm, num_sms, stream)  \
         : launch_stream<W, H, false, __nv_bfloat16>(ta, tb, tsa, tsb, ta, ta, prm, num_sms, stream))
    if (wide) return halves == 2 ? MXP_S_LAUNCH(true, 2) : MXP_S_LAUNCH(true, 1);
    return halves == 2 ? MXP_S_LAUNCH(false, 2) : MXP_S_LAUNCH(false, 1);
#undef MXP_S_LAUNCH
}

// ------------------------------------------------------------------------------ sparse residual
int stream_b_form(mxp_mode a_mode, mxp_mode b_mode)
{
    const bool one_sided = (a_mode == MXP_MODE_MXFP4_PLUS && b_mode == MXP_MODE_MXFP4) ||
                           (a_mode == MXP_MODE_MXFP4 && b_mode == MXP_MODE_MXFP4_PLUS);
    if (one_sided && override_get(MXP_KNOB_ONE_SIDED) != 1)
        return b_mode == MXP_MODE_MXFP4_PLUS ? MXP_PREPACK_SPLIT : MXP_PREPACK_PLAIN;
    return (a_mode != MXP_MODE_MXFP4 || b_mode != MXP_MODE_MXFP4) ? stream_wide_form(b_mode) : MXP_PREPACK_PLAIN;
}

// One operand MXFP4+, the other MXFP4 (see the head of this file).  0: not supported.
size_t stream_sparse_workspace_bytes(int64_t M, int64_t N, int64_t K, mxp_mode a_mode, mxp_mode b_mode,
                                     bool b_prepacked)
{
    const bool ap = a_mode == MXP_MODE_MXFP4_PLUS, bp = b_mode == MXP_MODE_MXFP4_PLUS;
    if (ap == bp || (ap ? b_mode : a_mode) != MXP_MODE_MXFP4) return 0;
    if (M <= 128 || N <= 128 || K < 128 || K % 128 != 0) return 0;
    if ((uint64_t)M * (uint64_t)K / 16 >= (1ull << 32) || (uint64_t)N * (uint64_t)K / 16 >= (1ull << 32))
        return 0;
    const int64_t rows_x = ap ? M : N, rows_y = ap ? N : M;
    return sparse_layout(rows_x, rows_y, K, b_prepacked && bp, b_prepacked && ap).total;
}

// Where a quantizer that prepares an MXFP4+ A for the sparse-residual GEMM itself has to write
// inside the workspace of a call with a prepacked (plain MXFP4) B.
bool stream_a_split_layout(int64_t M, int64_t K, size_t* atoms, size_t* main, size_t* res, size_t* meta,
                           size_t* meta_pad_offset, size_t* meta_pad_bytes, size_t* total)
{
    if (M <= 128 || K < 256 || K % 256 != 0 || (uint64_t)M * (uint64_t)K / 16 >= (1ull << 32)) return false;
    const SparseLayout l = sparse_layout(M, 0, K, false, true);
    const SplitLayout lx = split_layout(M, K);
    *atoms = l.x + lx.atoms;
    *main = l.x + lx.main;
    *res = l.x + lx.res;
    *meta = l.x + lx.meta;
    // row groups (of 128 rows) that reach past row M: their blocks are contiguous at the end
    const size_t rgs = (size_t)row_groups(M, kTileM), full = (size_t)(M / 128), stages = (size_t)(K / 256);
    *meta_pad_offset = full * stages * 2048;
    *meta_pad_bytes = (rgs - full) * stages * 2048;
    *total = l.total;
    return true;
}

// `a_ready`: A (the MXFP4+ side) has been split into the workspace by the quantizer, which also
// cleared the status block; needs a prepacked B, so that nothing is left to prepare.
mxp_status launch_gemm_tc_sparse(int64_t M, int64_t N, int64_t K, const mxp_packed& A, const mxp_packed& B,
                                 const void* b_prepacked, void* D, mxp_dtype d_dt, int64_t ldd,
                                 void* workspace, size_t workspace_bytes, cudaStream_t stream, bool a_ready)
{
    if (a_ready && (b_prepacked == nullptr || A.mode != MXP_MODE_MXFP4_PLUS || K % 256 != 0)) return MXP_ERR_UNSUPPORTED;
    const size_t need = stream_sparse_workspace_bytes(M, N, K, A.mode, B.mode, b_prepacked != nullptr);
    if (need == 0) return MXP_ERR_UNSUPPORTED;
    if (workspace == nullptr || workspace_bytes < need) return MXP_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) || (reinterpret_cast<uintptr_t>(b_prepacked) & 255))
        return MXP_ERR_INVALID_ARG;
    // X: the MX+ operand, in the instruction's A slot; Y: the plain one.  X = B: D^T = B A^T.
    const bool swap = B.mode == MXP_MODE_MXFP4_PLUS;
    const mxp_packed& X = swap ? B : A;
    const mxp_packed& Y = swap ? A : B;
    const int64_t rows_x = X.rows, rows_y = Y.rows;
    if (((reinterpret_cast<uintptr_t>(X.nibbles) | reinterpret_cast<uintptr_t>(Y.nibbles)) & 15) ||
        ((reinterpret_cast<uintptr_t>(X.scales) | reinterpret_cast<uintptr_t>(Y.scales)) & 3))
        return MXP_ERR_INVALID_ARG;
    const int num_sms = sm_count();
    if (num_sms <= 0) return MXP_ERR_CUDA;
    const bool x_pre = swap && b_prepacked != nullptr, y_pre = !swap && b_prepacked != nullptr;
    const SparseLayout l = sparse_layout(rows_x, rows_y, K, x_pre, y_pre);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int kgroups = (int)(K / 128);
    const int halves = choose_halves(rows_x, rows_y, false, num_sms);
    const int sub = sub_n(false, halves);
    const int rgx = (int)row_groups(rows_x, kTileM), rgy = (int)row_groups(rows_y, sub);
    const uint8_t* x_base = x_pre ? static_cast<const uint8_t*>(b_prepacked) : ws + l.x;
    const SplitLayout lx = split_layout(rows_x, K);
    const uint8_t* y_atoms =
        y_pre ? static_cast<const uint8_t*>(b_prepacked) + packed_layout(rows_y, K, 0).atoms[halves - 1]
              : ws + l.y;
    const PrepackOperand px = (x_pre || a_ready) ? no_operand() : split_operand(X, ws + l.x);
    const PrepackOperand py =
        y_pre ? no_operand() : prepack_operand(Y, rows_y, K, false, sub, ws + l.y, nullptr);
    const uint64_t ctas = (uint64_t)px.scale_ctas + py.scale_ctas + px.split_ctas;
    if ((ctas == 0 && !a_ready) || ctas > 0x7FFFFFFFull) return MXP_ERR_UNSUPPORTED;
    if (ctas != 0) {
        prepack_kernel<<<(unsigned)ctas, 256, 0, stream>>>(px, py, static_cast<StatusBlock*>(workspace));
        if (cudaGetLastError() != cudaSuccess) return MXP_ERR_CUDA;
    }

    CUtensorMap ta, tb, tsa, tsb, tres, tmeta;
    const bool maps_ok = make_tmap_rows(&ta, x_base + lx.main, rows_x, K / 2, 128) &&
                         make_tmap_rows(&tb, Y.nibbles, rows_y, K / 2, sub / 2) &&
                         make_tmap_atoms(&tsa, x_base + lx.atoms, rgx, kgroups, 2, 1) &&
                         make_tmap_atoms(&tsb, y_atoms, rgy, kgroups, 2, 2 * halves) &&
                         make_tmap_rows64(&tres, x_base + lx.res, rows_x, K / 4) &&
                         make_tmap_meta(&tmeta, x_base + lx.meta, rgx, (K + 255) / 256);
    if (!maps_ok) return MXP_ERR_CUDA;
    SParams prm;
    prm.M = (int)rows_x;
    prm.N = (int)rows_y;
    prm.K = (int)K;
    prm.a_fmt = prm.b_fmt = 0;
    prm.parts_a = prm.parts_b = 1;
    prm.D = D;
    prm.ldd = ldd;
    prm.d_vec_ok = !swap && ((reinterpret_cast<uintptr_t>(D) & 15) == 0) &&
                   ((ldd * (d_dt == MXP_BF16 ? 2 : 4)) % 16 == 0);
    prm.transposed = swap ? 1 : 0;
    prm.status = static_cast<StatusBlock*>(workspace);
    const bool f32 = d_dt == MXP_F32;
    if (halves == 2)
        return f32 ? launch_stream<false, 2, true, float>(ta, tb, tsa, tsb, tres, tmeta, prm, num_sms, stream)
                   : launch_stream<false, 2, true, __nv_bfloat16>(ta, tb, tsa, tsb, tres, tmeta, prm, num_sms, stream);
    return f32 ? launch_stream<false, 1, true, float>(ta, tb, tsa, tsb, tres, tmeta, prm, num_sms, stream)
               : launch_stream<false, 1, true, __nv_bfloat16>(ta, tb, tsa, tsb, tres, tmeta, prm, num_sms, stream);
}

}  // namespace mxp
