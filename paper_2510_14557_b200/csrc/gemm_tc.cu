// Block-scaled FP4 tensor-core GEMM on MXFP4 / MXFP4+ operands (sm_100a).
//
//   D[M,N] = dec(A)[M,K] * dec(B)[N,K]^T, fp32 accumulation in tensor memory.
//
// Data path per K tile of 256 elements: TMA brings 128-byte rows of packed nibbles into a
// 128B-swizzled shared-memory ring; "aux" threads (one per operand row) gather the E8M0
// scale bytes into the 32x16-byte atoms tcgen05.cp wants and, for MX+ operands, patch the
// block-max nibbles in place; one elected thread issues tcgen05.mma kind::mxf4.block_scale.
//
// MX+ on FP4 tensor cores follows the paper's Eq. 4 / Algorithm 1: the BM value
// 4 + m/2 (E2M3-like) is split into BM_H = 4 + 2*m2 and BM_L = m1 + m0/2, both valid E2M1.
// The main tile gets BM_H in place of the BM nibble (ReplaceBM); a second tile that is zero
// except for BM_L at the BM positions (MakeFragment) goes through an extra MMA into the same
// accumulator.  With both operands in MX+ the product expands into four passes.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdio>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mxp {
namespace {

constexpr int BM = 128;             // rows of A per tile
constexpr int BK = 256;             // elements of K per stage = 128 bytes of nibbles
constexpr int kRowBytes = BK / 2;   // 128
constexpr int kAuxThreads = 128;
constexpr int kThreads = 64 + kAuxThreads;  // warp 0: TMA, warp 1: MMA, warps 2..5: aux + epilogue
constexpr long long kWaitLimit = 4000000000ll;  // cycles (~2 s) before a wait gives up
constexpr uint32_t kTmemCols = 512;

template <int BN, bool AP, bool BP>
struct Cfg {
    static constexpr int kATile = BM * kRowBytes;  // 16 KB
    static constexpr int kBTile = BN * kRowBytes;
    static constexpr int kStageData = kATile * (AP ? 2 : 1) + kBTile * (BP ? 2 : 1);
    static constexpr int kSfA = 2 * 512;               // two K groups of 128
    static constexpr int kSfB = (BN / 128) * 2 * 512;  // per 128 rows, two K groups
    static constexpr int kPrev = (AP ? BM * 8 : 0) + (BP ? BN * 8 : 0);  // idx bytes of last use
    static constexpr int kStageAux = kSfA + kSfB + kPrev;
    static constexpr int kBudget = 220 * 1024;
    static constexpr int kStagesRaw = (kBudget - 1024) / (kStageData + kStageAux);
    static constexpr int kStages = kStagesRaw > 8 ? 8 : kStagesRaw;
    static constexpr int kSmem = kStages * (kStageData + kStageAux) + 1024 /*barriers*/ + 1024 /*align*/;
    static_assert(kStages >= 2, "not enough shared memory for two stages");
};

struct Params {
    int M, N, K;
    const uint8_t* a_scales;
    const uint8_t* a_index;
    const uint8_t* b_scales;
    const uint8_t* b_index;
    void* D;
    int64_t ldd;
    int d_vec_ok;  // D rows are 16-byte aligned: the epilogue may use 128-bit stores
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

// Offset of byte column c (0..127) of row r inside a 128B-swizzled tile.
__device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t c)
{
    return r * 128u + ((((c >> 4) ^ (r & 7u)) << 4) | (c & 15u));
}

// Loads the 8 scale (or index) bytes of one row for the K tile starting at block j0.
// K % 128 == 0, so the row holds a multiple of four bytes and words are 4-byte aligned.
__device__ __forceinline__ uint2 load_row_bytes(const uint8_t* plane, int64_t row, int rows,
                                                int nbk, int j0, uint32_t fill)
{
    uint2 v = make_uint2(fill, fill);
    if (plane != nullptr && row < rows) {
        const uint32_t* p = reinterpret_cast<const uint32_t*>(plane + row * (int64_t)nbk + j0);
        if (j0 < nbk) v.x = __ldg(p);
        if (j0 + 4 < nbk) v.y = __ldg(p + 1);
    }
    return v;
}

// ReplaceBM / MakeFragment for one operand row and K tile, in shared memory.
//   hi: the TMA-written tile; lo: the residual tile (zero outside BM positions).
__device__ __forceinline__ void patch_row(uint8_t* hi, uint8_t* lo, uint32_t r, uint2 idx,
                                          uint2 sc, int nblocks)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t ib = ((j < 4 ? idx.x : idx.y) >> (8 * (j & 3))) & 31u;
        const uint32_t sb = ((j < 4 ? sc.x : sc.y) >> (8 * (j & 3))) & 255u;
        if (j < nblocks && sb != 0u) {
            const uint32_t off = swz(r, 16u * j + (ib >> 1));
            const uint32_t b = hi[off];
            const uint32_t n = (ib & 1u) ? (b >> 4) : (b & 15u);
            const uint32_t h = (n & 8u) | 6u | ((n >> 2) & 1u);  // BM_H: E2M1 code 11 m2
            const uint32_t l = (n & 8u) | (n & 3u);              // BM_L: E2M1 code 0 m1 m0
            hi[off] = (uint8_t)((ib & 1u) ? ((b & 0x0Fu) | (h << 4)) : ((b & 0xF0u) | h));
            lo[off] = (uint8_t)((ib & 1u) ? (l << 4) : l);
        }
    }
}
__device__ __forceinline__ void clear_row(uint8_t* lo, uint32_t r, uint2 idx)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t ib = ((j < 4 ? idx.x : idx.y) >> (8 * (j & 3))) & 31u;
        lo[swz(r, 16u * j + (ib >> 1))] = 0;
    }
}

template <int BN, bool AP, bool BP, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const Params prm)
{
    using C = Cfg<BN, AP, BP>;
    constexpr int S = C::kStages;
    constexpr int kBRowsPerThread = BN / kAuxThreads;  // 1 or 2

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~(uintptr_t)1023);
    // layout: [S x stage data][S x stage aux][barriers]
    uint8_t* data0 = smem;
    uint8_t* aux0 = smem + S * C::kStageData;
    uint64_t* bars = reinterpret_cast<uint64_t*>(aux0 + S * C::kStageAux);
    uint64_t* full = bars;            // TMA bytes landed
    uint64_t* ready = bars + S;       // aux threads done (scales staged, BM patched)
    uint64_t* empty = bars + 2 * S;   // MMAs that read the stage have completed
    uint64_t* acc_full = bars + 3 * S;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * S + 1);
    volatile uint32_t* abort = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);

    auto a_hi = [&](int s) { return data0 + s * C::kStageData; };
    auto b_hi = [&](int s) { return data0 + s * C::kStageData + C::kATile; };
    auto a_lo = [&](int s) { return data0 + s * C::kStageData + C::kATile + C::kBTile; };
    auto b_lo = [&](int s) {
        return data0 + s * C::kStageData + C::kATile + C::kBTile + (AP ? C::kATile : 0);
    };
    auto sfa = [&](int s) { return aux0 + s * C::kStageAux; };
    auto sfb = [&](int s) { return aux0 + s * C::kStageAux + C::kSfA; };
    auto prev_a = [&](int s) { return aux0 + s * C::kStageAux + C::kSfA + C::kSfB; };
    auto prev_b = [&](int s) {
        return aux0 + s * C::kStageAux + C::kSfA + C::kSfB + (AP ? BM * 8 : 0);
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int nbk = prm.K / 32;
    const int ktiles = (prm.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&ready[s], kAuxThreads);
            ptx::mbar_init(&empty[s], 1);
        }
        ptx::mbar_init(acc_full, 1);
        *abort = 0u;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_a);
        ptx::prefetch_tmap(&tmap_b);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }
    if (AP || BP) {
        // residual tiles start as all zero
        for (int s = 0; s < S; ++s) {
            if (AP)
                for (int i = threadIdx.x; i < C::kATile / 16; i += kThreads)
                    reinterpret_cast<uint4*>(a_lo(s))[i] = make_uint4(0, 0, 0, 0);
            if (BP)
                for (int i = threadIdx.x; i < C::kBTile / 16; i += kThreads)
                    reinterpret_cast<uint4*>(b_lo(s))[i] = make_uint4(0, 0, 0, 0);
        }
        ptx::fence_proxy_async_smem();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_acc = tmem_base;             // BN columns of fp32
    const uint32_t tmem_sfa = tmem_base + BN;        // 4 columns per K group, 2 groups
    const uint32_t tmem_sfb = tmem_base + BN + 8;    // BN/32 columns per K group, 2 groups

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int kt = 0; kt < ktiles; ++kt) {
                const int s = kt % S;
                const uint32_t use = kt / S;
                if (use > 0 && !ptx::mbar_wait(&empty[s], (use - 1) & 1, abort, kWaitLimit)) {
                    give_up(abort, prm.status, 0x100 + s);
                    break;
                }
                ptx::mbar_arrive_expect_tx(&full[s], C::kATile + C::kBTile);
                ptx::tma_load_2d(a_hi(s), &tmap_a, &full[s], kt * kRowBytes, m0);
                ptx::tma_load_2d(b_hi(s), &tmap_b, &full[s], kt * kRowBytes, n0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t accumulate = 0;
            bool ok = true;
            for (int kt = 0; kt < ktiles && ok; ++kt) {
                const int s = kt % S;
                const uint32_t ph = (kt / S) & 1;
                if (!ptx::mbar_wait(&full[s], ph, abort, kWaitLimit) ||
                    !ptx::mbar_wait(&ready[s], ph, abort, kWaitLimit)) {
                    give_up(abort, prm.status, 0x200 + s);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint64_t da_hi = ptx::smem_desc_sw128(ptx::smem_u32(a_hi(s)));
                const uint64_t db_hi = ptx::smem_desc_sw128(ptx::smem_u32(b_hi(s)));
                const uint64_t da_lo = AP ? ptx::smem_desc_sw128(ptx::smem_u32(a_lo(s))) : 0;
                const uint64_t db_lo = BP ? ptx::smem_desc_sw128(ptx::smem_u32(b_lo(s))) : 0;
                const int groups = (prm.K - kt * BK) >= BK ? 2 : 1;  // K % 128 == 0
                for (int g = 0; g < groups; ++g) {
                    const uint32_t t_sfa = tmem_sfa + 4 * g;
                    const uint32_t t_sfb = tmem_sfb + (BN / 32) * g;
                    ptx::tc_cp_sf(t_sfa, ptx::smem_desc_sf(ptx::smem_u32(sfa(s) + 512 * g)));
#pragma unroll
                    for (int h = 0; h < BN / 128; ++h)
                        ptx::tc_cp_sf(t_sfb + 4 * h,
                                      ptx::smem_desc_sf(ptx::smem_u32(sfb(s) + 1024 * h + 512 * g)));
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        // 64 elements = 32 bytes per MMA: advance the start address field
                        const uint64_t adv = (uint64_t)((g * 2 + kk) * 32 >> 4);
                        const uint32_t idesc =
                            ptx::idesc_block_scaled(1, 1, BM, BN, 2 * kk, 2 * kk);
                        ptx::mma_mxf4(tmem_acc, da_hi + adv, db_hi + adv, idesc, t_sfa, t_sfb,
                                      accumulate);
                        accumulate = 1;
                        if (AP)
                            ptx::mma_mxf4(tmem_acc, da_lo + adv, db_hi + adv, idesc, t_sfa, t_sfb, 1);
                        if (BP)
                            ptx::mma_mxf4(tmem_acc, da_hi + adv, db_lo + adv, idesc, t_sfa, t_sfb, 1);
                        if (AP && BP)
                            ptx::mma_mxf4(tmem_acc, da_lo + adv, db_lo + adv, idesc, t_sfa, t_sfb, 1);
                    }
                }
                ptx::tc_commit(&empty[s]);
            }
            if (ok) ptx::tc_commit(acc_full);
        }
    } else {
        // ------------------------------------------------------------------ aux threads
        const int t = threadIdx.x - 64;  // 0..127: A row t, B rows t (+128)
        const int64_t arow = (int64_t)m0 + t;
        bool ok = true;
        uint2 sa = load_row_bytes(prm.a_scales, arow, prm.M, nbk, 0, 0u);
        uint2 ia = AP ? load_row_bytes(prm.a_index, arow, prm.M, nbk, 0, 0u) : make_uint2(0, 0);
        uint2 sbv[kBRowsPerThread], ibv[kBRowsPerThread];
#pragma unroll
        for (int h = 0; h < kBRowsPerThread; ++h) {
            const int64_t brow = (int64_t)n0 + t + 128 * h;
            sbv[h] = load_row_bytes(prm.b_scales, brow, prm.N, nbk, 0, 0u);
            ibv[h] = BP ? load_row_bytes(prm.b_index, brow, prm.N, nbk, 0, 0u) : make_uint2(0, 0);
        }
        const uint32_t sf_off = (uint32_t)(t & 31) * 16u + (uint32_t)(t >> 5) * 4u;
        for (int kt = 0; kt < ktiles && ok; ++kt) {
            const int s = kt % S;
            const uint32_t use = kt / S;
            // prefetch the next tile's bytes while this one is processed
            const int jn = (kt + 1) * 8;
            const uint2 sa_n = load_row_bytes(prm.a_scales, arow, prm.M, nbk, jn, 0u);
            const uint2 ia_n = AP ? load_row_bytes(prm.a_index, arow, prm.M, nbk, jn, 0u)
                                  : make_uint2(0, 0);
            uint2 sb_n[kBRowsPerThread], ib_n[kBRowsPerThread];
#pragma unroll
            for (int h = 0; h < kBRowsPerThread; ++h) {
                const int64_t brow = (int64_t)n0 + t + 128 * h;
                sb_n[h] = load_row_bytes(prm.b_scales, brow, prm.N, nbk, jn, 0u);
                ib_n[h] = BP ? load_row_bytes(prm.b_index, brow, prm.N, nbk, jn, 0u)
                             : make_uint2(0, 0);
            }
            if (use > 0 && !ptx::mbar_wait(&empty[s], (use - 1) & 1, abort, kWaitLimit)) {
                give_up(abort, prm.status, 0x300 + s);
                ok = false;
                break;
            }
            // scale atoms: row r -> 16-byte line r % 32, word r / 32; one atom per K group
            *reinterpret_cast<uint32_t*>(sfa(s) + sf_off) = sa.x;
            *reinterpret_cast<uint32_t*>(sfa(s) + 512 + sf_off) = sa.y;
#pragma unroll
            for (int h = 0; h < kBRowsPerThread; ++h) {
                *reinterpret_cast<uint32_t*>(sfb(s) + 1024 * h + sf_off) = sbv[h].x;
                *reinterpret_cast<uint32_t*>(sfb(s) + 1024 * h + 512 + sf_off) = sbv[h].y;
            }
            if (AP || BP) {
                if (use > 0) {  // undo the residual nibbles of the stage's previous use
                    if (AP)
                        clear_row(a_lo(s), t, *reinterpret_cast<const uint2*>(prev_a(s) + t * 8));
                    if (BP)
#pragma unroll
                        for (int h = 0; h < kBRowsPerThread; ++h)
                            clear_row(b_lo(s), t + 128 * h,
                                      *reinterpret_cast<const uint2*>(prev_b(s) + (t + 128 * h) * 8));
                }
                if (!ptx::mbar_wait(&full[s], use & 1, abort, kWaitLimit)) {
                    give_up(abort, prm.status, 0x400 + s);
                    ok = false;
                    break;
                }
                const int nblocks = min(8, nbk - kt * 8);
                if (AP) {
                    if (arow < prm.M) patch_row(a_hi(s), a_lo(s), t, ia, sa, nblocks);
                    // rows beyond M and blocks beyond K leave nothing to clear next time:
                    // remember index bytes only where a patch may have been written
                    *reinterpret_cast<uint2*>(prev_a(s) + t * 8) = ia;
                }
                if (BP) {
#pragma unroll
                    for (int h = 0; h < kBRowsPerThread; ++h) {
                        const int64_t brow = (int64_t)n0 + t + 128 * h;
                        if (brow < prm.N)
                            patch_row(b_hi(s), b_lo(s), t + 128 * h, ibv[h], sbv[h], nblocks);
                        *reinterpret_cast<uint2*>(prev_b(s) + (t + 128 * h) * 8) = ibv[h];
                    }
                }
            }
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(&ready[s]);
            sa = sa_n;
            ia = ia_n;
#pragma unroll
            for (int h = 0; h < kBRowsPerThread; ++h) {
                sbv[h] = sb_n[h];
                ibv[h] = ib_n[h];
            }
        }

        // ------------------------------------------------------------------ epilogue
        if (ok && !ptx::mbar_wait(acc_full, 0, abort, kWaitLimit)) {
            give_up(abort, prm.status, 0x500);
            ok = false;
        }
        if (ok) {
            ptx::tc_fence_after_sync();
            const int q = warp & 3;  // TMEM lane quarter this warp may read
            const int row = m0 + 32 * q + lane;
            OutT* drow = static_cast<OutT*>(prm.D) + (int64_t)row * prm.ldd + n0;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(tmem_acc + ((uint32_t)(32 * q) << 16) + 32 * c, r);
                ptx::tmem_ld_wait();
                const int col0 = n0 + 32 * c;
                if (row < prm.M && col0 < prm.N) {
                    if (col0 + 32 <= prm.N && prm.d_vec_ok) {
                        if (sizeof(OutT) == 4) {
                            uint4* p = reinterpret_cast<uint4*>(drow + 32 * c);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                p[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
                        } else {
                            uint32_t w[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(
                                    __uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                                w[i] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            uint4* p = reinterpret_cast<uint4*>(drow + 32 * c);
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                p[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
                        }
                    } else {
                        for (int i = 0; i < 32 && col0 + i < prm.N; ++i) {
                            if (sizeof(OutT) == 4)
                                reinterpret_cast<float*>(drow)[32 * c + i] = __uint_as_float(r[i]);
                            else
                                reinterpret_cast<__nv_bfloat16*>(drow)[32 * c + i] =
                                    __float2bfloat16_rn(__uint_as_float(r[i]));
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    // After a give-up the producer may still have copies in flight: let them land (bounded)
    // before the CTA's shared memory goes away.
    if (*abort != 0u && threadIdx.x == 0) {
        const long long t0 = clock64();
        for (int s = 0; s < S; ++s)
            while (!ptx::mbar_try_wait(&full[s], 0) && !ptx::mbar_try_wait(&full[s], 1) &&
                   clock64() - t0 < kWaitLimit) {
            }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------ host side
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                              const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                              const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn()
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

// Packed nibbles as a 2-D byte tensor [rows][K/2], boxes of 128 bytes x box_rows, 128B swizzle.
bool make_tmap(CUtensorMap* m, const uint8_t* base, int64_t rows, int64_t K, int box_rows)
{
    EncodeFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
    const cuuint32_t box[2] = {(cuuint32_t)kRowBytes, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, bool AP, bool BP, typename OutT>
mxp_status launch_cfg(const CUtensorMap& ta, const CUtensorMap& tb, const Params& prm,
                      cudaStream_t stream)
{
    using C = Cfg<BN, AP, BP>;
    auto kern = gemm_tc_kernel<BN, AP, BP, OutT>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmem) !=
            cudaSuccess)
            return MXP_ERR_CUDA;
        attr_set = true;
    }
    dim3 grid((unsigned)((prm.M + BM - 1) / BM), (unsigned)((prm.N + BN - 1) / BN));
    kern<<<grid, kThreads, C::kSmem, stream>>>(ta, tb, prm);
    return cudaGetLastError() == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

template <int BN, typename OutT>
mxp_status launch_modes(bool ap, bool bp, const CUtensorMap& ta, const CUtensorMap& tb,
                        const Params& prm, cudaStream_t stream)
{
    if (ap && bp) return launch_cfg<BN, true, true, OutT>(ta, tb, prm, stream);
    if (ap) return launch_cfg<BN, true, false, OutT>(ta, tb, prm, stream);
    if (bp) return launch_cfg<BN, false, true, OutT>(ta, tb, prm, stream);
    return launch_cfg<BN, false, false, OutT>(ta, tb, prm, stream);
}

}  // namespace

size_t tc_workspace_bytes(int64_t, int64_t, int64_t, mxp_mode, mxp_mode) { return kStatusBytes; }

mxp_status launch_gemm_tc(int64_t M, int64_t N, int64_t K, const mxp_packed& A,
                          const mxp_packed& B, void* D, mxp_dtype d_dt, int64_t ldd,
                          void* workspace, size_t, cudaStream_t stream)
{
    if (K % 128 != 0) return MXP_ERR_UNSUPPORTED;
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return MXP_ERR_UNSUPPORTED;
    if ((N + 127) / 128 > 65535) return MXP_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(A.scales) & 3) || (reinterpret_cast<uintptr_t>(B.scales) & 3))
        return MXP_ERR_INVALID_ARG;
    const bool ap = A.mode == MXP_MODE_MXFP4_PLUS, bp = B.mode == MXP_MODE_MXFP4_PLUS;
    if ((ap && (reinterpret_cast<uintptr_t>(A.bm_index) & 3)) ||
        (bp && (reinterpret_cast<uintptr_t>(B.bm_index) & 3)))
        return MXP_ERR_INVALID_ARG;
    const int bn = (N > 128) ? 256 : 128;
    CUtensorMap ta, tb;
    if (!make_tmap(&ta, A.nibbles, M, K, BM) || !make_tmap(&tb, B.nibbles, N, K, bn))
        return MXP_ERR_CUDA;
    Params prm;
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.a_scales = A.scales;
    prm.a_index = A.bm_index;
    prm.b_scales = B.scales;
    prm.b_index = B.bm_index;
    prm.D = D;
    prm.ldd = ldd;
    prm.d_vec_ok = ((reinterpret_cast<uintptr_t>(D) & 15) == 0) &&
                   ((ldd * (d_dt == MXP_BF16 ? 2 : 4)) % 16 == 0);
    prm.status = static_cast<StatusBlock*>(workspace);
    if (cudaMemsetAsync(workspace, 0, sizeof(StatusBlock), stream) != cudaSuccess)
        return MXP_ERR_CUDA;
    if (d_dt == MXP_F32)
        return bn == 256 ? launch_modes<256, float>(ap, bp, ta, tb, prm, stream)
                         : launch_modes<128, float>(ap, bp, ta, tb, prm, stream);
    return bn == 256 ? launch_modes<256, __nv_bfloat16>(ap, bp, ta, tb, prm, stream)
                     : launch_modes<128, __nv_bfloat16>(ap, bp, ta, tb, prm, stream);
}

mxp_status tensor_peak_probe(int, int, double*, double*) { return MXP_ERR_UNSUPPORTED; }

}  // namespace mxp
