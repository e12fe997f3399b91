// Weight-only GEMM for decode shapes (1 <= M <= 16) on the FP4 tensor path:
//
//   D[M,N] = A(bf16)[M,K] * dec(W)[N,K]^T          (Sec. 7.1 setting; decode per Eq. 3)
//
// The operation is bound by streaming the weights once (0.5625 bytes per element), so the
// design removes everything else from the path of the bytes:
//   * tcgen05.mma kind::mxf4 reads packed E2M1 codes with one E8M0 scale per 32 elements, which
//     is how the weights are stored: no thread ever touches a weight.
//   * The weights are re-tiled ONCE (decode_prepack_kernel; a re-ordering of the 4-bit codes,
//     not a dequantization): every CTA owns a fixed range of weight rows, and what it needs for
//     256 elements of K -- its rows' codes in the 128-byte-swizzled order the MMA reads, their
//     scales in the 32-lane atoms tcgen05.cp copies, the BM records -- is one contiguous piece
//     of about 11 KB that a single cp.async.bulk brings in.  148 CTAs read 148 sequential
//     streams.  The rows are dealt out evenly, a CTA on every SM (decode_plan says why).
//   * MX+ (Eq. 4): the re-tiled codes hold BM_H (4 or 6, an E2M1 value) in the BM's place; the
//     rest, BM_L in {0, 0.5, 1, 1.5}, also E2M1, goes into a second operand tile that is zero
//     elsewhere, built per stage from one record byte per block (position, BM_L, sign) by four
//     warps, and multiplied by a second MMA into the same accumulator with the same scales.
//   * The bf16 activations become FP4 as well: per block of 32 the magnitudes, 13 bits below
//     the block's largest exponent, are written in balanced base 8 (five digits -4..3), each
//     digit plane an operand row of E2M1 values 0..4 with its own block scale 2^(E - 3 j); the
//     epilogue adds the planes' accumulator columns.  An element within 2^5 of its block's
//     maximum is exact, a smaller one is rounded at 2^-13 of that maximum's binade.
//     A small kernel does this once per call (decode_act_kernel) and leaves the operand images
//     of all stages in the workspace; the GEMM is launched as its programmatic dependent, so
//     its CTAs stream weights meanwhile, and fetches the images stage by stage next to the
//     weights.  (Converting inside the GEMM, every CTA for itself, costs a CTA 0.5-0.9 us per
//     activation row -- ~280 instructions per eight elements, sixteen warps' worth per row --
//     which from the fourth row on is more than the second launch costs in a chain.)
//   * Up to three activation rows (kSelf; two with MX+ weights): the dependent chain "kernel
//     before -> conversion kernel -> this kernel's copies of the images" costs more than the
//     conversion itself.  There every CTA converts the rows for itself, straight into shared
//     memory where the images of all stages stay (40 KB at K = 4096: three rows' planes fill
//     one 16-row operand tile), while its weights are already streaming: one launch per call,
//     and no image travels through global memory.  The number of rows is a template argument.
//     MX+ there takes Eq. 4's BM_L term off the tensor cores: sum over blocks of
//     (+-BM_L 2^shared_exp) a[k_BM] is eight products per weight row and stage, so warps 10-21
//     add it on the CUDA cores in fp32 from the record bytes, the scale bytes and a raw bf16
//     copy of the activations in shared memory -- one thread per weight row, the eight weights
//     built without a branch and the eight activations fetched by independent loads (a form
//     with a thread per (row, block) and the loads behind one another was ~3x slower and lost
//     to the extra MMAs).  No BM_L tile is built and the MMA count per stage is that of plain
//     MXFP4; the epilogue adds the groups' partial sums in a fixed order.
//   * Set-up order (each step measured with per-phase time stamps): warp 0 initialises the
//     barriers, a lane per ring slot, and issues the first ring-full of weight copies; sixteen
//     bulk-copy instructions take that warp ~0.5 us, so it only arrives at the set-up barrier
//     and nobody waits for it.  With kSelf the other warps ask for the activations before
//     anything else: a load from L2 issued once the weight stream is running queues behind it
//     (~1 us instead of ~0.3).  A stage's four scale copies go out ahead of its four MMAs.
//   * warp 0 issues the weight copies,
//     warp 1 the activation copies, warps 2-5 the MMAs (each every fourth stage, with an
//     accumulator of its own), warps 6-9 drain the accumulators, warps 10-21 handle BM_L:
//     for M >= 2 they build the BM_L operand tiles (four groups of three, group g owning slot g
//     of the tile ring: one group needs ~1 us per stage, the stream delivers one every
//     0.26 us), for self-converted rows they sum the term themselves (the same grouping where
//     a tile has at most 96 rows, else three groups of four; a stage each in turn).
//   * A call may name the weights of the call expected next: once its own have all but
//     landed, a CTA asks for the head of its share of them into L2 (the last MMAs, the switch
//     to the next call's CTAs and their first copies' latency move no weights otherwise).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mxp {
namespace {

constexpr int kIssueWarp0 = 2, kIssuers = 4;
constexpr int kRowWarp0 = 6;
constexpr int kResWarp0 = 10;  // the first of the twelve warps that handle BM_L
constexpr int kTileWarps = 3, kTileGroups = 4;  // ... as four groups of three (tiles for M >= 4, sums below)
constexpr int kWarps = kResWarp0 + kTileWarps * kTileGroups;
constexpr int kThreads = 32 * kWarps;
constexpr int kStageK = 256;   // elements of K per stage: 128 bytes of codes per row
constexpr int kPlanes = 5;     // balanced base-8 digit planes of an activation
constexpr int kMaxM = 16;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemSf = 384;  // scale-factor columns: 16 per issuer
constexpr int kAtom = 512;
constexpr int kMaxStages = 16;
constexpr long long kWaitLimit = 4000000000ll;
constexpr size_t kSmemMax = 227 * 1024;
constexpr size_t kActSpread = 116 * 1024;  // shared memory that only one CTA per SM can have
constexpr int kHintLead = 2;               // images still in flight when the hint for the next call goes out
constexpr size_t kHintBytes = 192 * 1024;  // what a CTA asks for of the next call's weights (a ring-full)
constexpr uint32_t kMagic = 0x4D58D0C2u;
}  // namespace
constexpr size_t kHeaderBytes = 256;
namespace {

// Rows of the activation operand: five planes per activation row, padded to the MMA's N.
__host__ __device__ constexpr int act_rows(int M) { return (kPlanes * M + 15) / 16 * 16; }
__host__ __device__ constexpr int sfb_bytes(int nact) { return (nact < 32 ? nact : 32) * 16; }
__host__ __device__ constexpr size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// How the weight rows are dealt out: a function of the shape and of the SM count only, so the
// one-off re-tiling and every later call agree.
struct DecodePlan {
    int rows;      // weight rows per tile at most (<= 128): what an image has room for
    int tiles;     // tiles per CTA
    int ctas;
    int nst;       // stages of kStageK per tile
    int base, extra;  // tile j (= CTA * tiles + tile of the CTA) holds base + (j < extra) rows
    uint32_t wimg;  // bytes of one (CTA, tile, stage) weight image
};
// First weight row of tile j and the number of rows it holds.
__host__ __device__ inline int64_t tile_row0(int64_t j, int base, int extra)
{
    return j * base + (j < extra ? j : (int64_t)extra);
}
__host__ __device__ inline int tile_rows(int64_t j, int base, int extra, int64_t N)
{
    const int64_t r0 = tile_row0(j, base, extra);
    int64_t r = base + (j < extra ? 1 : 0);
    if (r0 + r > N) r = N - r0;
    return r > 0 ? (int)r : 0;
}
__host__ inline bool decode_plan(int64_t N, int64_t K, bool plus, int sms, DecodePlan* p)
{
    if (N < 1 || K < kStageK || K % kStageK != 0 || K > 32768 || sms < 1 || N > (1ll << 30)) return false;
    p->tiles = (int)((N + (int64_t)sms * 128 - 1) / ((int64_t)sms * 128));
    // The rows are dealt out as evenly as they go, so that every SM has a CTA: an SM left
    // without one takes in as many CTAs of the small conversion kernel as it has room for
    // (seven of its sixteen), which then run one after another on that SM's issue slots while
    // the other 147 SMs wait for the last of them (measured: 4.6 us instead of 1).
    const int64_t T = (int64_t)sms * p->tiles;
    if (N / T >= 8) {
        p->base = (int)(N / T);
        p->extra = (int)(N % T);
        p->rows = p->base + (p->extra > 0 ? 1 : 0);
        p->ctas = sms;
    } else {  // few rows: tiles of eight, fewer CTAs
        p->base = p->rows = 8;
        p->extra = 0;
        p->ctas = (int)((N + 8 * (int64_t)p->tiles - 1) / (8 * (int64_t)p->tiles));
    }
    p->nst = (int)(K / kStageK);
    p->wimg = (uint32_t)up((size_t)p->rows * 128 + 2 * kAtom + (plus ? (size_t)p->rows * 8 : 0), 16);
    return true;
}

struct PrepackHeader {
    uint32_t magic, mode, rows, tiles, ctas, nst, wimg, pad;
    int64_t N, K;
};

// Shared memory of the GEMM kernel (bytes from the 1024-byte aligned base).
// Three rings.  The weight ring (`stages` slots of `slot` bytes) is as deep as the rest allows:
// the weights do not depend on the kernel before, so whatever fits streams in while the
// activations are still being waited for.  The activation images (from L2, available late,
// needed only just before their MMAs) and, for MX+, the BM_L tiles built from the weight
// images' records have rings of their own (`astages` slots of `aslot` bytes, kSideSlots slots of
// `rslot` bytes).
// kSelf form (self_nst > 0: number of stages whose activation images stay resident): no side
// rings; behind the weight ring come the images' code tiles (2 KB a stage), their scale atoms
// (512 bytes a stage) and, for MX+, the raw activations and the BM_L term's sums.
struct DecodeLayout {
    size_t slot, act0, aslot, res0, rslot, bars, total;
    size_t img_codes, img_sf, raw, corr;  // kSelf only (raw, corr: MX+)
    int stages, astages;
};
constexpr int kSelfMaxM = 3;  // rows the self-converting form takes: three rows' planes fill one 16-row operand tile
constexpr int kSideSlots = 4;
// kSelf: bytes between the code tiles of two stages.  The MMA's second group of eight operand
// rows lies 1024 bytes behind the first (the descriptor's stride).  A single activation row has
// five planes, so its second group holds nothing the epilogue looks at and may as well be the
// next stage's first group: a tile then costs 1 KB instead of 2 (plus one tile of room at the
// end), which lets the MXFP4+ form keep all sixteen stages of K = 4096 in its ring.
__host__ __device__ constexpr int self_img_bytes(int self_m) { return kPlanes * self_m <= 8 ? 1024 : 2048; }
__host__ __device__ inline DecodeLayout decode_layout(int rows, uint32_t wimg, int nact, bool plus, int stages,
                                                      int self_nst = 0, int astages = kSideSlots, int self_m = 1)
{
    DecodeLayout l;
    l.stages = stages;
    l.astages = astages;
    l.img_codes = l.img_sf = l.raw = l.corr = 0;
    l.act0 = l.aslot = l.res0 = l.rslot = 0;
    l.slot = up(wimg, 1024);
    if (self_nst > 0) {
        const size_t last = (size_t)(stages - 1) * l.slot + 128 * 128;  // (see below)
        size_t o = up(last > (size_t)stages * l.slot ? last : (size_t)stages * l.slot, 1024);
        l.img_codes = o;
        o += (size_t)(self_nst + 1) * self_img_bytes(self_m);
        l.img_sf = o;
        o += (size_t)self_nst * 512;
        if (plus) {
            l.raw = o;   // the activation rows as given (bf16), for the BM_L term
            o += (size_t)self_m * (size_t)self_nst * kStageK * 2;
            l.corr = o;  // its sums [group][row m][weight row]
            o += (size_t)kTileGroups * self_m * 128 * sizeof(float);
        }
        l.bars = up(o, 16);
        l.total = l.bars + 512 + 1024;  // barriers (under 512 bytes); slack for aligning the base
        return l;
    }
    l.act0 = (size_t)stages * l.slot;
    l.aslot = up((size_t)nact * 128 + 2 * (size_t)sfb_bytes(nact), 1024);
    l.res0 = l.act0 + (size_t)astages * l.aslot;
    l.rslot = plus ? up((size_t)rows * 128, 1024) : 0;
    // an MMA reads 128 rows of 128 bytes from the start of a tile that holds fewer: what follows
    // the last tile must exist (any bytes are finite E2M1 codes; the rows are never read back)
    size_t off = up(l.res0 + kSideSlots * l.rslot + 16384, 16);
    l.bars = off;
    l.total = off + 1024 + 1024;  // barriers; slack for aligning the base
    return l;
}

#ifdef MXP_DECODE_TIMELINE  // measurement build: per-CTA time stamps of the last launch, read back by a probe
// [CTA][event]: 32 + st = an issuer starts stage st; 54 = thread 64 has converted its share,
// 55 = warp 0 has issued its copies; 56 + p = phase p (MXP_TL: 0 entry, 1 set-up done,
// 2 activations available, 3 / 4 first / last stage seen by its issuer, 5 all MMAs done,
// 6 output stored).  A stamp is one store and nothing else: a form that first looked up
// which launch of a graph it belonged to (eight loads) held the stamping warp up by ~0.6 us
// and moved every phase behind it.
__device__ unsigned long long g_decode_tl2[256 * 64];
#define MXP_TL(slot) do { g_decode_tl2[blockIdx.x * 64 + 56 + (slot)] = ptx::globaltimer_ns(); } while (0)
#define MXP_TL2(ev) do { g_decode_tl2[blockIdx.x * 64 + (ev)] = ptx::globaltimer_ns(); } while (0)
// the conversion kernel's CTA c uses row 200 + c: 0 entry, 1 images cleared, 2 dependency wait over,
// 3 converted, 4 stored, 8 = the SM it ran on
#define MXP_TLA(ev) do { if (threadIdx.x == 0) g_decode_tl2[(200 + blockIdx.x) * 64 + (ev)] = ptx::globaltimer_ns(); } while (0)
#else
#define MXP_TL(slot) do { } while (0)
#define MXP_TL2(ev) do { } while (0)
#define MXP_TLA(ev) do { } while (0)
#endif


struct DecodeParams {
    int M, N;
    const __nv_bfloat16* A;  // kSelf: the activations, row stride lda
    int64_t lda;
    int clear_status;      // kSelf: this launch clears the status block (no kernel ahead of it does)
    const uint8_t* wimg;   // weight images [cta][tile][stage]
    const uint8_t* aimg;   // activation images [stage] (not kSelf)
    const uint8_t* next_wimg;  // weight images of the call expected next, or nullptr ...
    size_t next_share;         // ... and the bytes of them that belong to one CTA of this grid
    void* D;
    int64_t ldd;
    StatusBlock* status;   // may be nullptr
    int rows, tiles, nst, stages, astages;
    int base, extra;       // the split of the weight rows over the tiles (see DecodePlan)
    uint32_t wimg_bytes;
};

__device__ __forceinline__ void report(StatusBlock* st, volatile uint32_t* abort, uint32_t where)
{
    *abort = 1u;
    if (st != nullptr && atomicCAS(&st->code, 0u, (uint32_t)MXP_ERR_TIMEOUT) == 0u) st->where = where;
}

// Offset of 16-byte chunk c (0..7) of row r inside a 128B-swizzled tile.
__host__ __device__ __forceinline__ uint32_t swz_chunk(uint32_t r, uint32_t c)
{
    return r * 128u + ((c ^ (r & 7u)) << 4);
}

__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(ptx::smem_u32(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(ptx::smem_u32(bar))
        : "memory");
}

// ------------------------------------------------------------------------------------------
// One-off re-tiling of the weights.  grid (ctas * tiles, nst), 128 threads: thread r = row r
// of the tile.  Image of one (CTA, tile, stage):
//   [rows x 128 bytes of codes, 16-byte chunk c of row r at chunk c ^ (r & 7)]
//   [2 scale atoms of 512 bytes: byte of row r, block b at (r % 32) * 16 + (r / 32) * 4 + b % 4]
//   [MX+: rows x 8 record bytes: BM position | BM_L code << 5 | sign << 7; 0 = nothing to add]
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
decode_prepack_kernel(const uint8_t* __restrict__ nibbles, const uint8_t* __restrict__ scales,
                      const uint8_t* __restrict__ bm_index, int64_t N, int64_t K, int plus, int rows,
                      int base, int extra, uint32_t wimg, uint8_t* __restrict__ out, PrepackHeader hdr)
{
    const int r = threadIdx.x;
    const int64_t tile = blockIdx.x;
    const int st = blockIdx.y;
    if (tile == 0 && st == 0 && r == 0) *reinterpret_cast<PrepackHeader*>(out) = hdr;
    uint8_t* img = out + kHeaderBytes + ((size_t)tile * gridDim.y + st) * wimg;
    const int64_t n = tile_row0(tile, base, extra) + r;
    const bool live = r < tile_rows(tile, base, extra, N);
    uint4 code[8];
    uint8_t sc[8], rec[8];
#pragma unroll
    for (int kb = 0; kb < 8; ++kb) {
        code[kb] = make_uint4(0u, 0u, 0u, 0u);
        sc[kb] = 0x7F;
        rec[kb] = 0;
    }
    if (live) {
        const int64_t b0 = n * (K / 32) + (int64_t)st * 8;
#pragma unroll
        for (int kb = 0; kb < 8; ++kb) {
            code[kb] = __ldg(reinterpret_cast<const uint4*>(nibbles + (b0 + kb) * 16));
            sc[kb] = scales[b0 + kb];
            if (sc[kb] == 0) code[kb] = make_uint4(0u, 0u, 0u, 0u);  // flushed block: zeros
            if (plus && sc[kb] != 0 && sc[kb] != 0xFF) {
                const uint32_t pos = bm_index[b0 + kb] & 31u;
                uint32_t* w = &code[kb].x + (pos >> 3);  // (x, y, z, w are consecutive words)
                const uint32_t sh = (pos & 7u) * 4u;
                const uint32_t nib = (*w >> sh) & 15u;   // sign, m2 m1 m0
                const uint32_t hi = (nib & 8u) | 6u | ((nib >> 2) & 1u);  // BM_H: E2M1 code 11 m2
                *w = (*w & ~(15u << sh)) | (hi << sh);
                rec[kb] = (uint8_t)(pos | ((nib & 3u) << 5) | ((nib & 8u) << 4));
                if ((nib & 3u) == 0u) rec[kb] = 0;       // BM_L = 0
            }
        }
    }
    if (r < rows) {
#pragma unroll
        for (int kb = 0; kb < 8; ++kb)
            *reinterpret_cast<uint4*>(img + swz_chunk((uint32_t)r, (uint32_t)kb)) = code[kb];
        if (plus) {
            uint2 v;
            v.x = (uint32_t)rec[0] | ((uint32_t)rec[1] << 8) | ((uint32_t)rec[2] << 16) | ((uint32_t)rec[3] << 24);
            v.y = (uint32_t)rec[4] | ((uint32_t)rec[5] << 8) | ((uint32_t)rec[6] << 16) | ((uint32_t)rec[7] << 24);
            *reinterpret_cast<uint2*>(img + (size_t)rows * 128 + 2 * kAtom + (size_t)r * 8) = v;
        }
    }
    // every row of the atoms gets a finite scale, also those past the tile
    uint8_t* atoms = img + (size_t)rows * 128;
    const uint32_t so = (uint32_t)(r & 31) * 16u + (uint32_t)(r >> 5) * 4u;
    const bool use = r < rows;
    *reinterpret_cast<uint32_t*>(atoms + so) =
        use ? (uint32_t)sc[0] | ((uint32_t)sc[1] << 8) | ((uint32_t)sc[2] << 16) | ((uint32_t)sc[3] << 24) : 0x7F7F7F7Fu;
    *reinterpret_cast<uint32_t*>(atoms + kAtom + so) =
        use ? (uint32_t)sc[4] | ((uint32_t)sc[5] << 8) | ((uint32_t)sc[6] << 16) | ((uint32_t)sc[7] << 24) : 0x7F7F7F7Fu;
}

// Eight activations (quarter `qd` of block `kb` of a stage, activation row m; the four lanes of
// a quad hold the four quarters of one block) -> their five digit planes: one word of codes per
// plane into the stage's tile `codes`, and the planes' scale bytes into its atoms `sf`.
// (`codes`, `sf`: shared-memory addresses; the stores name the shared window, which saves the
// 64-bit address arithmetic of generic stores.)
__device__ __forceinline__ void convert_quarter(const uint4 v, int m, int kb, int qd, uint32_t codes, uint32_t sf,
                                                int sfb)
{
    const uint32_t x[4] = {v.x, v.y, v.z, v.w};
    // largest exponent field of the block (zero and subnormals count as field 1): both halves of
    // a register at once
    uint32_t e2 = 0x00010001u;
#pragma unroll
    for (int q = 0; q < 4; ++q) e2 = __vmaxu2(e2, (x[q] >> 7) & 0x00FF00FFu);
    uint32_t eb = max(e2 & 0xFFFFu, e2 >> 16);
    eb = max(eb, __shfl_xor_sync(0xFFFFFFFFu, eb, 1));
    eb = max(eb, __shfl_xor_sync(0xFFFFFFFFu, eb, 2));
    const bool nonfinite = eb == 255u;
    // t = |a| / 2^(E - 12), rounded to an integer below 2^13 (half up), plus 4 in each of five
    // octal places: octal digit j of t, minus 4, is the balanced digit d_j in -4..3 with
    // |a| = sum_j d_j 2^(E - 3 j).  The scaling is a multiply by a power of two (exact), the
    // rounding an add of one half and a truncating conversion (the sum is exact wherever the
    // truncation could depend on it).  2^(12 - E) has exponent field 266 - eb: beyond 254 (blocks
    // below 2^-115) it is applied in two steps.
    const uint32_t fld = 266u - eb, f1 = min(fld, 254u);
    const float s1 = __uint_as_float(f1 << 23), s2 = __uint_as_float((127u + fld - f1) << 23);
    uint32_t p[4];  // two elements per register
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float lo = __uint_as_float((x[q] << 16) & 0x7FFF0000u) * s2;
        const float hi = __uint_as_float(x[q] & 0x7FFF0000u) * s2;
        p[q] = (__float2uint_rz(fmaf(lo, s1, 0.5f)) | (__float2uint_rz(fmaf(hi, s1, 0.5f)) << 16)) + 0x49244924u;
    }
    // per plane: the octal digits of four elements as the four selector nibbles of one byte
    // permute, which looks the digits' E2M1 codes up in an eight-byte table (codes of 4 3 2 1 0 1
    // 2 3, the sign bit set for the negative digits 0..3); an element's own sign is
    // exclusive-ored on top
    const uint32_t sg0 = __byte_perm((x[0] >> 12) & 0x00080008u, (x[1] >> 12) & 0x00080008u, 0x6420);
    const uint32_t sg1 = __byte_perm((x[2] >> 12) & 0x00080008u, (x[3] >> 12) & 0x00080008u, 0x6420);
    constexpr uint32_t kLutLo = 0x0A0C0D0Eu, kLutHi = 0x05040200u;
    const uint32_t row0 = (uint32_t)(kPlanes * m);
    const uint32_t sf0 = sf + (uint32_t)((kb >> 2) * sfb + (kb & 3));
#pragma unroll
    for (int j = 0; j < kPlanes; ++j) {
        const int sbyte = (int)eb - 3 * j;  // E8M0 byte of 2^(E - 3 j)
        const int sh = 3 * (4 - j);
        const uint32_t d0 = __byte_perm((p[0] >> sh) & 0x00070007u, (p[1] >> sh) & 0x00070007u, 0x6420);
        const uint32_t d1 = __byte_perm((p[2] >> sh) & 0x00070007u, (p[3] >> sh) & 0x00070007u, 0x6420);
        const uint32_t n0 = d0 | (d0 >> 4), n1 = d1 | (d1 >> 4);  // bytes 0 and 2: two digits each
        const uint32_t c0 = __byte_perm(kLutLo, kLutHi, __byte_perm(n0, 0u, 0x4420)) ^ sg0;
        const uint32_t c1 = __byte_perm(kLutLo, kLutHi, __byte_perm(n1, 0u, 0x4420)) ^ sg1;
        const uint32_t y0 = c0 | (c0 >> 4), y1 = c1 | (c1 >> 4);  // bytes 0 and 2: two codes each
        // a plane whose scale would lie below the format's range, or a block with an Inf or NaN: zeros
        const uint32_t w = (sbyte >= 0 && !nonfinite) ? __byte_perm(y0, y1, 0x6420) : 0u;
        const uint32_t row = row0 + (uint32_t)j;
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(codes + swz_chunk(row, (uint32_t)kb) + 4u * (uint32_t)qd), "r"(w)
                     : "memory");
        if (qd == 0)
            asm volatile("st.shared.u8 [%0], %1;" ::"r"(sf0 + (row & 31u) * 16u + (row >> 5) * 4u),
                         "r"(nonfinite ? 255u : (uint32_t)max(sbyte, 0))
                         : "memory");
    }
}

// ------------------------------------------------------------------------------------------
// Activations -> FP4 digit planes, once per call.  grid nst, 32 * M threads (four per block of
// 32 elements, eight elements each).  Image of one stage:
//   [nact rows x 128 bytes of codes, swizzled as above; row 5 m + j = plane j of activation m]
//   [2 scale atoms of sfb_bytes(nact): byte of row n, block b at (n % 32) * 16 + (n / 32) * 4 + b % 4]
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32 * kMaxM)
decode_act_kernel(const __nv_bfloat16* __restrict__ A, int64_t lda, int M, int nact, uint8_t* __restrict__ aimg,
                  StatusBlock* status, int clear_status)
{
    MXP_TLA(0);
#ifdef MXP_DECODE_TIMELINE
    if (threadIdx.x == 0) {
        unsigned sm;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
        g_decode_tl2[(200 + blockIdx.x) * 64 + 8] = sm;
    }
#endif
    ptx::grid_launch_dependents();  // the GEMM's CTAs may start streaming weights now
    extern __shared__ uint8_t img[];  // nact * 128 + 2 * sfb
    const int st = blockIdx.x;
    const int sfb = sfb_bytes(nact);
    const int bytes = nact * 128 + 2 * sfb;
    for (int i = threadIdx.x; i < nact * 128 / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(img)[i] = make_uint4(0u, 0u, 0u, 0u);   // absent rows: zero codes ...
    for (int i = threadIdx.x; i < 2 * sfb / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(img + nact * 128)[i] = make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);
    __syncthreads();  // ... with a finite scale; the rows in use land on top
    MXP_TLA(1);
    ptx::grid_dependency_wait();  // A may come from the kernel before
    MXP_TLA(2);
    if (clear_status && st == 0 && threadIdx.x == 0 && status != nullptr) {
        status->code = 0u;
        status->where = 0u;
    }
    const int i = threadIdx.x, blk = i >> 2, qd = i & 3;
    const int m = blk >> 3, kb = blk & 7;
    if (m < M) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(A + (int64_t)m * lda + (int64_t)st * kStageK + kb * 32) + qd);
        convert_quarter(v, m, kb, qd, ptx::smem_u32(img), ptx::smem_u32(img + nact * 128), sfb);
    }
    __syncthreads();
    MXP_TLA(3);
    uint4* dst = reinterpret_cast<uint4*>(aimg + (size_t)st * bytes);
    for (int k = threadIdx.x; k < bytes / 16; k += blockDim.x) dst[k] = reinterpret_cast<const uint4*>(img)[k];
    MXP_TLA(4);
}

// ------------------------------------------------------------------------------------------
// The GEMM.  kNact: rows of the activation operand (16 .. 80); kPlus: MXFP4+ weights.
// ------------------------------------------------------------------------------------------
// kSelfM: 0 = the activation images come from the conversion kernel; 1..3 = that many
// activation rows, converted by every CTA for itself (a literal, so that the planes' addresses fold).
template <int kNact, bool kPlus, int kSelfM, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_decode_tc_kernel(const DecodeParams prm)
{
    constexpr bool kSelf = kSelfM > 0;
    constexpr int kSelfRows = kSelf ? kSelfM : 1;
    static_assert(kSelfM <= kSelfMaxM && kPlanes * kSelfMaxM <= 16, "self-converted rows share one 16-row tile");
    static_assert(!kSelf || kNact == 16, "self-converted activations: one operand tile of 16 rows");
    constexpr int kSfb = sfb_bytes(kNact);
    constexpr int kMt = kSelf ? kSelfRows : kNact / kPlanes;  // activation rows the operand can hold
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int S = prm.stages;
    const int nst = prm.nst;
    const DecodeLayout L = decode_layout(prm.rows, prm.wimg_bytes, kNact, kPlus, S, kSelf ? nst : 0, prm.astages, kSelfRows);
    const int SA = prm.astages;  // slots of the activation ring
    // (what the kSelf form uses comes first and stays under the 512 bytes its layout reserves)
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);  // the slot's weight image landed
    uint64_t* empty = full + kMaxStages;       // the slot's MMAs are done (and its records read)
    uint64_t* acc_full = empty + kMaxStages;
    uint64_t* acc_empty = acc_full + 1;
    uint64_t* corr_full = acc_empty + 1;       // kSelf MX+: a tile's BM_L sums are complete
    uint64_t* corr_empty = corr_full + 1;      // ... and have been taken
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(corr_empty + 1);
    volatile uint32_t* abort = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);
    static_assert((2 * kMaxStages + 4) * 8 + 8 <= 384, "barriers of the kSelf form");
    uint64_t* afull = reinterpret_cast<uint64_t*>(smem + L.bars + 384);  // the slot's activation image landed
    uint64_t* aempty = afull + kMaxStages;     // its MMAs are done
    uint64_t* res_full = aempty + kMaxStages;  // [kSideSlots] the slot's BM_L tile is written
    uint64_t* res_empty = res_full + kSideSlots;  //           its MMAs are done
    static_assert(384 + (2 * kMaxStages + 2 * kSideSlots) * 8 <= 1024, "barriers of the three-ring form");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // kSelf, MX+: the twelve BM_L warps as four groups of three (a thread per weight row, up to 96)
    // or, for taller tiles, three groups of four
    const int sum_warps = prm.rows <= 32 * kTileWarps ? kTileWarps : 4, sum_groups = 12 / sum_warps;
    auto slot = [&](int s) { return smem + (size_t)s * L.slot; };
    auto act_slot = [&](int sa) { return smem + L.act0 + (size_t)sa * L.aslot; };
    auto res_slot = [&](int sr) { return smem + L.res0 + (size_t)sr * L.rslot; };
    const int64_t tile0 = (int64_t)blockIdx.x * prm.tiles;  // first tile of this CTA
    // tiles of this CTA that hold rows, and its stages in all
    int ntl = 0;
    while (ntl < prm.tiles && tile_rows(tile0 + ntl, prm.base, prm.extra, prm.N) > 0) ++ntl;
    const uint32_t total = (uint32_t)(ntl * nst);
    const uint8_t* wsrc = prm.wimg + (size_t)blockIdx.x * prm.tiles * nst * prm.wimg_bytes;

    // ---------------------------------------------------------------------- set-up
    // Warp 0: barriers (a lane per ring slot), then the first ring-full of weight copies, a lane
    // each: the weights do not depend on the kernel before, and everything else overlaps their
    // latency.  Issuing sixteen bulk copies takes the warp ~0.5 us, so it only ARRIVES at the
    // set-up barrier (before the copies) and the other warps do not wait for it.
    // kSelf, warps 2 and up: the activations are asked for first of all (A is in stream order
    // after the wait; once the weight stream is running, a load from L2 queues behind it).
    constexpr int kConv0 = 64, kConv = kThreads - kConv0;  // threads that convert activations
    const int cid = (int)threadIdx.x - kConv0;
    const int per_row = kSelf ? nst * 32 : 0;  // eight-element pieces of a row: a thread takes piece i of every row
    auto fetch = [&](int m, int i) {
        return __ldg(reinterpret_cast<const uint4*>(prm.A + (int64_t)m * prm.lda + (int64_t)i * 8));
    };
    uint4 v[kSelfRows];
#pragma unroll
    for (int m = 0; m < kSelfRows; ++m) v[m] = make_uint4(0u, 0u, 0u, 0u);
    if (warp == 0) {
        if (lane == 0) MXP_TL(0);  // kernel entry
        if (lane < kMaxStages) {
            if (!kSelf) {
                ptx::mbar_init(&afull[lane], 1);
                ptx::mbar_init(&aempty[lane], 1);
            }
            ptx::mbar_init(&full[lane], 1);
            ptx::mbar_init(&empty[lane], !kPlus ? 1 : kSelf ? 1 + sum_warps : 1 + kTileWarps);  // + the warps that read its records
        } else if (lane < kMaxStages + kSideSlots) {
            if (!kSelf) {
                ptx::mbar_init(&res_full[lane - kMaxStages], kTileWarps);
                ptx::mbar_init(&res_empty[lane - kMaxStages], 1);
            }
        } else if (lane == kMaxStages + kSideSlots) {
            ptx::mbar_init(acc_full, kIssuers);
            ptx::mbar_init(acc_empty, 4);
            ptx::mbar_init(corr_full, kTileWarps * kTileGroups);
            ptx::mbar_init(corr_empty, 4);
            *abort = 0u;
        }
        ptx::fence_mbar_init();
        __threadfence_block();
        ptx::named_bar_arrive(1, kThreads);
        __syncwarp();
        const uint32_t c = (uint32_t)lane;
        if (c < total && c < (uint32_t)S) {
            ptx::mbar_arrive_expect_tx(&full[c], prm.wimg_bytes);
            bulk_g2s(slot((int)c), wsrc + (size_t)c * prm.wimg_bytes, prm.wimg_bytes, &full[c]);
        }
        if (lane == 0) MXP_TL2(55);
    } else {
        if (warp == 1) {
            ptx::tmem_alloc(tmem_slot, kTmemCols);
            ptx::tmem_relinquish();
        } else if (kSelf) {
            ptx::grid_dependency_wait();
            if (cid < per_row) {
#pragma unroll
                for (int m = 0; m < kSelfRows; ++m) v[m] = fetch(m, cid);
            }
            // the images' unused rows: zero codes under a finite scale (the rows in use land on top)
            for (int i = cid; i < (nst + 1) * (self_img_bytes(kSelfRows) / 16); i += kConv)
                reinterpret_cast<uint4*>(smem + L.img_codes)[i] = make_uint4(0u, 0u, 0u, 0u);
            for (int i = cid; i < nst * 32; i += kConv)
                reinterpret_cast<uint4*>(smem + L.img_sf)[i] =
                    make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);
        }
        ptx::tc_fence_before_sync();
        ptx::named_bar_sync(1, kThreads);
        ptx::tc_fence_after_sync();
    }
    ptx::grid_launch_dependents();  // whatever follows on the stream may be scheduled
    if (cid == 0) MXP_TL(1);  // set-up done
    if (kSelf) {
        // Activations -> digit planes, by this CTA for itself: a quad of lanes per block of 32,
        // eight elements per lane, straight into the resident images.
        if (prm.clear_status && blockIdx.x == 0 && cid == 0 && prm.status != nullptr) {
            prm.status->code = 0u;
            prm.status->where = 0u;
        }
        // (a thread's next eight elements are on their way from L2 while it converts these)
        const uint32_t img_codes0 = ptx::smem_u32(smem + L.img_codes), img_sf0 = ptx::smem_u32(smem + L.img_sf);
        int i = cid >= 0 ? cid : per_row;
        while (i < per_row) {
            const int nxt = i + kConv;
            uint4 vn[kSelfRows];
#pragma unroll
            for (int m = 0; m < kSelfRows; ++m) vn[m] = nxt < per_row ? fetch(m, nxt) : make_uint4(0u, 0u, 0u, 0u);
            const int st = i >> 5, kb = (i >> 2) & 7, qd = i & 3;
#pragma unroll
            for (int m = 0; m < kSelfRows; ++m) {
                if (kPlus) *reinterpret_cast<uint4*>(smem + L.raw + ((size_t)m * nst * kStageK + (size_t)i * 8) * 2) = v[m];
                convert_quarter(v[m], m, kb, qd, img_codes0 + (uint32_t)st * (uint32_t)self_img_bytes(kSelfRows), img_sf0 + (uint32_t)st * 512u, kSfb);
                v[m] = vn[m];
            }
            i = nxt;
        }
        if (cid == 0) MXP_TL2(54);
        ptx::fence_proxy_async_smem();  // the MMAs read the images through the async proxy
        ptx::tc_fence_before_sync();
        __syncthreads();
        ptx::tc_fence_after_sync();
        if (cid == 0) MXP_TL(2);  // activations available
    }
    const uint32_t tmem_base = *tmem_slot;  // (warp 0 of the form without this barrier does not use it)

    if (warp == 0) {
        // ---------------------------------------------------------------- weight copies (the rest)
        if (lane == 0) {
            for (uint32_t c = (uint32_t)S; c < total; ++c) {
                const int s = c % S;
                if (!ptx::mbar_wait(&empty[s], (c / S - 1) & 1, abort, kWaitLimit)) {
                    report(prm.status, abort, 0x7100 + s);
                    break;
                }
                ptx::mbar_arrive_expect_tx(&full[s], prm.wimg_bytes);
                bulk_g2s(slot(s), wsrc + (size_t)c * prm.wimg_bytes, prm.wimg_bytes, &full[s]);
            }
        }
        if (prm.next_wimg != nullptr && total > 0u) {
            // HBM has nothing to do from about here until the next call's CTAs have the SMs and
            // their first copies are out (~2.5 us of a ~6.8 us call): once all but this CTA's last
            // two images have landed, ask for the head of the next call's weights into L2, as much
            // as a CTA's ring holds.  (cp.async.bulk.prefetch.L2: a hint, nothing waits for it.)
            const uint32_t last = total > (uint32_t)kHintLead ? total - 1u - (uint32_t)kHintLead : 0u;
            if (lane == 0) ptx::mbar_wait(&full[last % S], (last / S) & 1, abort, kWaitLimit);
            __syncwarp();
            const size_t head = prm.next_share < kHintBytes ? prm.next_share : kHintBytes;
            const size_t piece = (head / 32 + 15) / 16 * 16;  // a lane each
            const size_t off = (size_t)lane * piece;
            if (*abort == 0u && piece > 0 && off < head) {
                const uint8_t* src = prm.next_wimg + (size_t)blockIdx.x * prm.next_share + off;
                const uint32_t n = (uint32_t)(head - off < piece ? head - off : piece);
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(n) : "memory");
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- activation copies
        if (!kSelf && lane == 0) {
            ptx::grid_dependency_wait();  // the activation images are the preceding kernel's output
            MXP_TL(2);  // activations available
            constexpr uint32_t kBytes = kNact * 128 + 2 * kSfb;
            for (uint32_t c = 0; c < total; ++c) {
                const int sa = c % SA;
                if (c >= (uint32_t)SA && !ptx::mbar_wait(&aempty[sa], (c / SA - 1) & 1, abort, kWaitLimit)) {
                    report(prm.status, abort, 0x7200 + sa);
                    break;
                }
                ptx::mbar_arrive_expect_tx(&afull[sa], kBytes);
                bulk_g2s(act_slot(sa), prm.aimg + (size_t)(c % (uint32_t)nst) * kBytes, kBytes, &afull[sa]);
            }
        }
    } else if (warp >= kIssueWarp0 && warp < kIssueWarp0 + kIssuers) {
        // ---------------------------------------------------------------- MMA issuers
        // Issuer i takes the stages whose running number is i (mod 4): the number of slots is a
        // multiple of four, so a slot always belongs to the same issuer, which sees every fill
        // of it in turn (the parity it waits for is never ambiguous).
        const int iss = warp - kIssueWarp0;
        const uint32_t tmem_acc = tmem_base + (uint32_t)(iss * kNact);
        uint32_t c = 0;
        bool ok = true;
        for (int t = 0; t < ntl && ok; ++t) {
            if (t > 0 && !ptx::mbar_wait(acc_empty, (uint32_t)(t - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x7300);
                break;
            }
            ptx::tc_fence_after_sync();
            const int first = (iss - (int)(c % kIssuers) + kIssuers) % kIssuers;
            for (int st = first; st < nst; st += kIssuers) {
                const uint32_t cc = c + (uint32_t)st;
                const int s = cc % S;
                const uint32_t ph = (cc / S) & 1;
                const int sa = kSelf ? 0 : cc % SA;                 // slot of the activation ring
                const int sd = cc % kSideSlots;                     // slot of the tile ring
                const uint32_t phd = (cc / kSideSlots) & 1;
                if (!ptx::mbar_wait(&full[s], ph, abort, kWaitLimit) ||
                    (!kSelf && !ptx::mbar_wait(&afull[sa], (cc / SA) & 1, abort, kWaitLimit))) {
                    if (lane == 0) report(prm.status, abort, 0x7400 + s);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
#ifdef MXP_DECODE_TIMELINE
                if (lane == 0 && st < 32) g_decode_tl2[blockIdx.x * 64 + 32 + st] = ptx::globaltimer_ns();
#endif
                if (lane == 0 && cc == 0) MXP_TL(3);          // first stage landed
                if (lane == 0 && cc == total - 1) MXP_TL(4);  // last stage landed
                const uint8_t* sl = slot(s);
                const uint64_t da = ptx::smem_desc_sw128(ptx::smem_u32(sl));
                const uint64_t db = ptx::smem_desc_sw128(
                    ptx::smem_u32(kSelf ? smem + L.img_codes + (size_t)st * self_img_bytes(kSelfRows) : act_slot(sa)));
                const uint32_t sfa = ptx::smem_u32(sl + (size_t)prm.rows * 128);
                const uint32_t sfb =
                    ptx::smem_u32(kSelf ? smem + L.img_sf + (size_t)st * 512 : act_slot(sa) + kNact * 128);
                const uint32_t t_sf = tmem_base + kTmemSf + 16u * (uint32_t)iss;
                if (ptx::elect_one()) {
#pragma unroll
                    for (int g = 0; g < 2; ++g) {  // 128 elements: one scale atom per operand
                        const uint32_t t_sfa = t_sf + 8u * (uint32_t)g, t_sfb = t_sfa + 4u;
                        ptx::tc_cp_sf(t_sfa, ptx::smem_desc_sf(sfa + (uint32_t)(g * kAtom)));
                        ptx::tc_cp_sf(t_sfb, ptx::smem_desc_sf(sfb + (uint32_t)(g * kSfb)));
                    }
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        const uint32_t t_sfa = t_sf + 8u * (uint32_t)g, t_sfb = t_sfa + 4u;
#pragma unroll
                        for (int kk = 0; kk < 2; ++kk) {  // 64 elements = 32 bytes per MMA
                            const uint64_t adv = (uint64_t)((g * 2 + kk) * 32 >> 4);
                            ptx::mma_mxf4(tmem_acc, da + adv, db + adv,
                                          ptx::idesc_block_scaled(1, 1, 128, kNact, 2 * kk, 2 * kk), t_sfa, t_sfb,
                                          (st == first && g == 0 && kk == 0) ? 0u : 1u);
                        }
                    }
                }
                __syncwarp();
                if (kPlus && !kSelf) {
                    // the BM_L tile of the stage, same scales, same accumulator (Eq. 4)
                    if (!ptx::mbar_wait(&res_full[sd], phd, abort, kWaitLimit)) {
                        if (lane == 0) report(prm.status, abort, 0x7500 + sd);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint64_t dr = ptx::smem_desc_sw128(ptx::smem_u32(res_slot(sd)));
                    if (ptx::elect_one()) {
#pragma unroll
                        for (int g = 0; g < 2; ++g) {
                            const uint32_t t_sfa = t_sf + 8u * (uint32_t)g, t_sfb = t_sfa + 4u;
#pragma unroll
                            for (int kk = 0; kk < 2; ++kk) {
                                const uint64_t adv = (uint64_t)((g * 2 + kk) * 32 >> 4);
                                ptx::mma_mxf4(tmem_acc, dr + adv, db + adv,
                                              ptx::idesc_block_scaled(1, 1, 128, kNact, 2 * kk, 2 * kk), t_sfa,
                                              t_sfb, 1u);
                            }
                        }
                    }
                    __syncwarp();
                }
                if (ptx::elect_one()) {  // the stage's slots are free once these MMAs have read them
                    ptx::tc_commit(&empty[s]);
                    if (!kSelf) ptx::tc_commit(&aempty[sa]);
                    if (kPlus && !kSelf) ptx::tc_commit(&res_empty[sd]);
                }
                __syncwarp();
            }
            c += (uint32_t)nst;
            if (!ok) break;
            if (ptx::elect_one()) ptx::tc_commit(acc_full);
            __syncwarp();
        }
    } else if (warp < kRowWarp0 + 4) {
        // ---------------------------------------------------------------- row warps (epilogue)
        // Thread = weight row of the tile = TMEM lane.  An output is the sum of its five planes'
        // columns over the four issuers' accumulators.
        const int q = warp & 3;  // the TMEM lane quarter this warp may read
        const int row = 32 * q + lane;
        ptx::grid_dependency_wait();  // D may still be in use by the kernel before
        for (int t = 0; t < ntl; ++t) {
            const int64_t n0 = tile_row0(tile0 + t, prm.base, prm.extra);
            const int rows_here = tile_rows(tile0 + t, prm.base, prm.extra, prm.N);
            if (!ptx::mbar_wait_relaxed(acc_full, (uint32_t)t & 1, abort, kWaitLimit, 200u)) {
                if (lane == 0) report(prm.status, abort, 0x7600);
                break;
            }
            ptx::tc_fence_after_sync();
            if (warp == kRowWarp0 && lane == 0 && t == ntl - 1) MXP_TL(5);  // all MMAs done
            float o[kMt];
#pragma unroll
            for (int m = 0; m < kMt; ++m) o[m] = 0.f;
            const uint32_t c0 = (uint32_t)t * (uint32_t)nst;
#pragma unroll
            for (int ch = 0; ch < kNact / 16; ++ch) {
                float part[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) part[j] = 0.f;
#pragma unroll
                for (int a = 0; a < kIssuers; ++a) {
                    // issuer a wrote its accumulator only if it had a stage of this tile
                    if ((a - (int)(c0 % kIssuers) + kIssuers) % kIssuers >= nst) continue;
                    uint32_t r2[16];
                    ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(a * kNact + 16 * ch), r2);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) part[j] += __uint_as_float(r2[j]);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if ((16 * ch + j) / kPlanes < kMt) o[(16 * ch + j) / kPlanes] += part[j];
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty);
            if (kSelf && kPlus) {
                // Eq. 4's BM_L term of this tile, summed on the CUDA cores by the warps below
                if (!ptx::mbar_wait_relaxed(&corr_full[0], (uint32_t)t & 1, abort, kWaitLimit, 100u)) {
                    if (lane == 0) report(prm.status, abort, 0x7900);
                    break;
                }
                const float* corr =
                    reinterpret_cast<const float*>(smem + L.corr);
#pragma unroll
                for (int m = 0; m < kSelfRows; ++m) {
                    float c = 0.f;
#pragma unroll
                    for (int g = 0; g < sum_groups; ++g) c += corr[(g * kSelfRows + m) * 128 + row];  // fixed order
                    o[m] += c;
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&corr_empty[0]);
            }
            if (row < rows_here) {
#pragma unroll
                for (int m = 0; m < kMt; ++m) {
                    if (m < prm.M) {
                        const int64_t off = (int64_t)m * prm.ldd + n0 + row;
                        if (sizeof(OutT) == 4)
                            static_cast<float*>(prm.D)[off] = o[m];
                        else
                            static_cast<__nv_bfloat16*>(prm.D)[off] = __float2bfloat16_rn(o[m]);
                    }
                }
            }
        }
    } else if (kPlus && kSelf) {
        // ---------------------------------------------------------------- BM_L on the CUDA cores
        // Group g of three warps takes the stages whose running number is g (mod 4); thread =
        // weight row (tiles of more than 96 rows: three groups of four warps).  A stage gives a row eight
        // record bytes (BM position | BM_L code << 5 | sign << 7) and eight scale bytes: eight
        // weights (BM_L 2^shared_exp), eight activations fetched independently of one another,
        // eight FMAs per activation row.  No branch: an absent BM_L is a zero weight.
        // (The sums are bound by instruction issue, ~160 per row and stage.  Three groups of four
        // warps, a thread per row of up to 128, left the fourth warp of every group without rows
        // at config 3's 75 and one of the SM's four schedulers without work: 0.65 us per stage
        // and group, the last group done 1.3 us after the MMAs.)
        const int grp = (warp - kResWarp0) / sum_warps;
        const int r = (int)threadIdx.x - 32 * (kResWarp0 + grp * sum_warps);
        const uint32_t raw_sa = ptx::smem_u32(smem + L.raw), slot0_sa = ptx::smem_u32(smem), slot_bytes = (uint32_t)L.slot;
        const uint32_t so = (uint32_t)(r & 31) * 16u + (uint32_t)(r >> 5) * 4u;
        bool ok = true;
        for (int t = 0; t < ntl && ok; ++t) {
            float acc[kSelfRows] = {};
            const int first = (grp + 12 - (int)(((uint32_t)t * (uint32_t)nst) % (uint32_t)sum_groups)) % sum_groups;
            for (int st = first; st < nst; st += sum_groups) {
                const uint32_t c = (uint32_t)t * (uint32_t)nst + (uint32_t)st;
                const int s = c % S;
                if (!ptx::mbar_wait(&full[s], (c / S) & 1, abort, kWaitLimit)) {
                    if (lane == 0) report(prm.status, abort, 0x7700 + s);
                    ok = false;
                    break;
                }
                {
                    if (r < prm.rows) {
                        // (loads that name the shared window: as generic loads through pointers the
                        // compiler cannot place, each costs 64-bit address arithmetic and more latency)
                        const uint32_t atoms = slot0_sa + (uint32_t)s * slot_bytes + (uint32_t)prm.rows * 128u;
                        uint2 rec;
                        uint32_t sc_lo, sc_hi;
                        asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(rec.x), "=r"(rec.y) : "r"(atoms + 2u * kAtom + (uint32_t)r * 8u) : "memory");
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sc_lo) : "r"(atoms + so) : "memory");
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sc_hi) : "r"(atoms + kAtom + so) : "memory");
                        float w[8];
                        uint32_t k[8];
#pragma unroll
                        for (int kb = 0; kb < 8; ++kb) {
                            const uint32_t b = ((kb < 4 ? rec.x : rec.y) >> (8 * (kb & 3))) & 255u;
                            const uint32_t sc = ((kb < 4 ? sc_lo : sc_hi) >> (8 * (kb & 3))) & 255u;
                            // BM_L 2^(sc - 127) = (code / 2) 2^(sc - 127), the sign from the record
                            const float mag = (float)((b >> 5) & 3u) * 0.5f * __uint_as_float(sc << 23);
                            w[kb] = __uint_as_float(__float_as_uint(mag) | ((b & 0x80u) << 24));
                            k[kb] = raw_sa + 2u * ((uint32_t)st * kStageK + (uint32_t)kb * 32u + (b & 31u));
                        }
#pragma unroll
                        for (int m = 0; m < kSelfRows; ++m) {
                            if (m < prm.M) {
                                float a[8];
#pragma unroll
                                for (int kb = 0; kb < 8; ++kb) {
                                    uint32_t hw;
                                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(hw) : "r"(k[kb] + 2u * (uint32_t)(m * nst * kStageK)) : "memory");
                                    a[kb] = __uint_as_float(hw << 16);
                                }
#pragma unroll
                                for (int kb = 0; kb < 8; ++kb) acc[m] = fmaf(w[kb], a[kb], acc[m]);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&empty[s]);  // the slot's records have been read
            }
            if (!ok) break;
            // the sums of the tile before must have been taken before this tile's are written
            if (t >= 1 && !ptx::mbar_wait(&corr_empty[0], (uint32_t)(t - 1) & 1, abort, kWaitLimit)) {
                if (lane == 0) report(prm.status, abort, 0x7A00);
                break;
            }
            float* corr = reinterpret_cast<float*>(smem + L.corr) + (size_t)grp * kSelfRows * 128;
            // this group's share, zeros included; with three warps the rows from 96 on hold no weights
#pragma unroll
            for (int m = 0; m < kSelfRows; ++m) {
                corr[m * 128 + r] = acc[m];
                if (sum_warps == kTileWarps && r < 32) corr[m * 128 + 96 + r] = 0.f;
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&corr_full[0]);
        }
    } else if (kPlus) {
        // ---------------------------------------------------------------- BM_L tiles
        // Group g of three warps owns slot g of the tile ring and takes the stages whose running
        // number is g (mod 4), like issuer g: every barrier of the slot is waited on by one party
        // only, stage after stage, so a parity never stands for the wrong phase.
        static_assert(kTileGroups == kSideSlots && kTileGroups == kIssuers, "one owner per slot");
        const int grp = (warp - kResWarp0) / kTileWarps;
        const int r0 = (int)threadIdx.x - 32 * (kResWarp0 + grp * kTileWarps);
        for (uint32_t c = (uint32_t)grp; c < total; c += kTileGroups) {
            const int s = c % S, sr = grp;
            // the stage's records have landed, and the MMAs that read the tile's last contents are done
            if (!ptx::mbar_wait(&full[s], (c / S) & 1, abort, kWaitLimit) ||
                (c >= (uint32_t)kSideSlots &&
                 !ptx::mbar_wait(&res_empty[sr], (c / kSideSlots - 1) & 1, abort, kWaitLimit))) {
                if (lane == 0) report(prm.status, abort, 0x7700 + s);
                break;
            }
            // A thread writes whole rows: per block one 16-byte chunk, zero but for the nibble its
            // record byte names (stores and loads name the shared window).
            const uint32_t tile = ptx::smem_u32(res_slot(sr));
            const uint32_t recs = ptx::smem_u32(slot(s)) + (uint32_t)prm.rows * 128u + 2u * kAtom;
            for (int r = r0; r < prm.rows; r += 32 * kTileWarps) {
                uint2 rec;
                asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(rec.x), "=r"(rec.y) : "r"(recs + (uint32_t)r * 8u) : "memory");
#pragma unroll
                for (int kb = 0; kb < 8; ++kb) {
                    const uint32_t b = ((kb < 4 ? rec.x : rec.y) >> (8 * (kb & 3))) & 255u;
                    // code 0 m1 m0 with the sign on top (0 when the record is empty), at nibble `pos` of the chunk
                    const uint32_t pos = b & 31u;
                    const uint32_t nib = (b & 0x60u) ? (((b >> 5) & 3u) | ((b >> 4) & 8u)) : 0u;
                    const uint32_t v = nib << (4u * (pos & 7u));
                    const uint32_t wi = pos >> 3;
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(
                                     tile + (uint32_t)r * 128u + ((((uint32_t)kb) ^ ((uint32_t)r & 7u)) << 4)),
                                 "r"(wi == 0u ? v : 0u), "r"(wi == 1u ? v : 0u), "r"(wi == 2u ? v : 0u), "r"(wi == 3u ? v : 0u)
                                 : "memory");
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_arrive(&res_full[sr]);
                ptx::mbar_arrive(&empty[s]);  // the slot's records have been read
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncthreads();
    if (threadIdx.x == 0) MXP_TL(6);  // output stored
    if (*abort != 0u && threadIdx.x == 0) {
        // after a timeout, copies may still be in flight into this CTA's shared memory: give
        // them (bounded) time to land before the CTA leaves
        const long long t0 = clock64();
        for (int s = 0; s < S; ++s)
            while (!ptx::mbar_try_wait(&full[s], 0) && !ptx::mbar_try_wait(&full[s], 1) &&
                   clock64() - t0 < kWaitLimit) {
            }
        for (int s = 0; s < SA && !kSelf; ++s)
            while (!ptx::mbar_try_wait(&afull[s], 0) && !ptx::mbar_try_wait(&afull[s], 1) &&
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

// Ring slots that fit: a multiple of four (see the issuers), at most sixteen.  self_nst > 0: the
// form with resident activation images.
int pick_stages(const DecodePlan& p, int nact, bool plus, int self_nst = 0, int astages = kSideSlots, int self_m = 1,
                int most = kMaxStages)
{
    for (int s = most; s >= 4; s -= 4)
        if (decode_layout(p.rows, p.wimg, nact, plus, s, self_nst, astages, self_m).total <= kSmemMax) return s;
    return 0;
}

template <int kNact, bool kPlus, int kSelfM, typename OutT>
cudaError_t launch(const DecodeParams& prm, int ctas, size_t smem, bool dependent, cudaStream_t stream)
{
    auto kern = gemm_decode_tc_kernel<kNact, kPlus, kSelfM, OutT>;
    static SmemAttrOnce once;
    cudaError_t e = ensure_dynamic_smem(kern, (int)kSmemMax, once);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    // A grid that may start before the kernel ahead of it has finished: always behind this
    // library's own conversion kernel; behind a caller's kernel only on the caller's promise.
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, prm);
}

template <int kNact, int kSelfM>
cudaError_t launch_n(bool plus, bool f32, const DecodeParams& prm, int ctas, size_t smem, bool dependent,
                     cudaStream_t stream)
{
    if (plus)
        return f32 ? launch<kNact, true, kSelfM, float>(prm, ctas, smem, dependent, stream)
                   : launch<kNact, true, kSelfM, __nv_bfloat16>(prm, ctas, smem, dependent, stream);
    return f32 ? launch<kNact, false, kSelfM, float>(prm, ctas, smem, dependent, stream)
               : launch<kNact, false, kSelfM, __nv_bfloat16>(prm, ctas, smem, dependent, stream);
}

}  // namespace

#ifdef MXP_DECODE_TIMELINE
extern "C" int mxp_decode_timeline_read2(unsigned long long* host, int n)
{
    return (int)cudaMemcpyFromSymbol(host, g_decode_tl2, sizeof(unsigned long long) * (size_t)n);
}
#endif

size_t decode_prepack_bytes(int64_t N, int64_t K, mxp_mode mode)
{
    if (mode != MXP_MODE_MXFP4 && mode != MXP_MODE_MXFP4_PLUS) return 0;
    DecodePlan p;
    if (!decode_plan(N, K, mode == MXP_MODE_MXFP4_PLUS, sm_count(), &p)) return 0;
    return kHeaderBytes + (size_t)p.ctas * p.tiles * p.nst * p.wimg;
}

size_t decode_workspace_bytes(int64_t M, int64_t K)
{
    if (M < 1 || M > kMaxM || K < kStageK || K % kStageK != 0 || K > 32768) return 0;
    const int nact = act_rows((int)M);
    return kStatusBytes + (size_t)(K / kStageK) * ((size_t)nact * 128 + 2 * (size_t)sfb_bytes(nact));
}

mxp_status decode_prepack(const mxp_packed& B, void* out, size_t out_bytes, cudaStream_t stream)
{
    const bool plus = B.mode == MXP_MODE_MXFP4_PLUS;
    DecodePlan p;
    if (!decode_plan(B.rows, B.cols, plus, sm_count(), &p)) return MXP_ERR_UNSUPPORTED;
    const size_t need = decode_prepack_bytes(B.rows, B.cols, B.mode);
    if (need == 0) return MXP_ERR_UNSUPPORTED;
    if (out == nullptr || out_bytes < need) return MXP_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(out) & 255) return MXP_ERR_INVALID_ARG;
    PrepackHeader h = {};
    h.magic = kMagic;
    h.mode = (uint32_t)B.mode;
    h.rows = (uint32_t)p.rows;
    h.tiles = (uint32_t)p.tiles;
    h.ctas = (uint32_t)p.ctas;
    h.nst = (uint32_t)p.nst;
    h.wimg = p.wimg;
    h.N = B.rows;
    h.K = B.cols;
    decode_prepack_kernel<<<dim3((unsigned)(p.ctas * p.tiles), (unsigned)p.nst), 128, 0, stream>>>(
        B.nibbles, B.scales, B.bm_index, B.rows, B.cols, plus ? 1 : 0, p.rows, p.base, p.extra, p.wimg,
        static_cast<uint8_t*>(out), h);
    return cudaGetLastError() == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

mxp_status launch_gemm_decode_tc(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, mxp_mode b_mode,
                                 const void* b_prepacked, size_t b_prepacked_bytes, void* D, mxp_dtype d_dt,
                                 int64_t ldd, void* workspace, size_t workspace_bytes, bool chained,
                                 const void* next_prepacked, size_t next_prepacked_bytes, cudaStream_t stream)
{
    const bool plus = b_mode == MXP_MODE_MXFP4_PLUS;
    DecodePlan p;
    if (M < 1 || M > kMaxM || !decode_plan(N, K, plus, sm_count(), &p)) return MXP_ERR_UNSUPPORTED;
    if (b_mode != MXP_MODE_MXFP4 && b_mode != MXP_MODE_MXFP4_PLUS) return MXP_ERR_UNSUPPORTED;
    // the re-tiled weights must be those of this shape, mode and device: their size says so
    if (b_prepacked_bytes != decode_prepack_bytes(N, K, b_mode)) return MXP_ERR_INVALID_ARG;
    const size_t need = decode_workspace_bytes(M, K);
    if (workspace == nullptr || workspace_bytes < need) return MXP_ERR_WORKSPACE;
    const int nact = act_rows((int)M);
    // up to three rows (one 16-row operand tile): every CTA converts them for itself, if the
    // images of all stages fit beside a ring.  (Measured at 11008 x 4096, chained: 7.7 / 8.1 us
    // for two / three rows against 8.6 / 8.8 us with the conversion kernel; with MX+ weights
    // 8.9 against 9.7 us for two rows, but 10.3 against 9.9 us for three: three rows as given
    // take 24 KB from the ring and triple the BM_L sums' gathers.)
    const bool try_self = M <= (plus ? 2 : kSelfMaxM);
    // (MX+, one row: with all sixteen stages of K = 4096 in the ring a call takes 8.1 us, with
    // twelve 7.6 us -- the CTAs of a call then finish closer together; why is not understood.
    // With the next call's weights on their way into L2 it is the other way round, 7.2 against
    // 7.6 us.  So: twelve unless there is a hint; a CTA with more than sixteen stages needs the
    // deeper ring either way.)
    const int most = (plus && M == 1 && next_prepacked == nullptr && p.tiles * p.nst <= kMaxStages) ? 12 : kMaxStages;
    const int self_stages = try_self ? pick_stages(p, nact, plus, p.nst, kSideSlots, (int)M, most) : 0;
    const bool self = self_stages != 0;
    // The activation ring: eight slots (the images come from L2 with ~1 us of latency: with four,
    // every fourth stage waits for its image) unless that leaves the weight ring fewer than eight.
    int astages = 2 * kSideSlots;
    if (self || pick_stages(p, nact, plus, 0, astages) < 8) astages = kSideSlots;
    const int stages = self ? self_stages : pick_stages(p, nact, plus, 0, astages);
    if (stages == 0) return MXP_ERR_UNSUPPORTED;
    const DecodeLayout L = decode_layout(p.rows, p.wimg, nact, plus, stages, self ? p.nst : 0, astages, self ? (int)M : 1);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    DecodeParams prm = {};
    prm.M = (int)M;
    prm.N = (int)N;
    prm.A = static_cast<const __nv_bfloat16*>(A);
    prm.lda = lda;
    prm.clear_status = chained ? 0 : 1;
    prm.wimg = static_cast<const uint8_t*>(b_prepacked) + kHeaderBytes;
    prm.aimg = ws + kStatusBytes;
    // the hint: every CTA asks for the head of "its" share of the weights expected next (with a
    // CTA on every SM in both calls that share is the next call's CTA's own stream)
    prm.next_wimg = nullptr;
    prm.next_share = 0;
    // (two self-converted rows against MX+ weights are the one case measured slower with it: 8.85
    // against 8.47 us)
    if (next_prepacked != nullptr && next_prepacked_bytes > kHeaderBytes && !(self && plus && M > 1)) {
        const size_t share = (next_prepacked_bytes - kHeaderBytes) / (size_t)p.ctas / 16 * 16;
        if (share >= 16) {
            prm.next_wimg = static_cast<const uint8_t*>(next_prepacked) + kHeaderBytes;
            prm.next_share = share;
        }
    }
    prm.D = D;
    prm.ldd = ldd;
    prm.status = reinterpret_cast<StatusBlock*>(ws);
    prm.rows = p.rows;
    prm.base = p.base;
    prm.extra = p.extra;
    prm.tiles = p.tiles;
    prm.nst = p.nst;
    prm.stages = stages;
    prm.astages = astages;
    prm.wimg_bytes = p.wimg;
    const bool f32 = d_dt == MXP_F32;
    if (self) {  // one launch; a programmatic dependent only on the caller's promise
        const cudaError_t e = M == 1   ? launch_n<16, 1>(plus, f32, prm, p.ctas, L.total, chained, stream)
                              : M == 2 ? launch_n<16, 2>(plus, f32, prm, p.ctas, L.total, chained, stream)
                                       : launch_n<16, 3>(plus, f32, prm, p.ctas, L.total, chained, stream);
        return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
    }
    {   // activations -> digit planes; in a chain it may start while the kernel before drains
        // (same shared-memory carve-out as the GEMM, so that the SMs are not reconfigured
        // between the two kernels of every call: that alone cost 1.6 us per call)
        static SmemAttrOnce carve;
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64 && !carve.done[dev]) {
            cudaFuncSetAttribute(decode_act_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared);
            if (cudaFuncSetAttribute(decode_act_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kActSpread) != cudaSuccess)
                return MXP_ERR_CUDA;
            carve.done[dev] = true;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)p.nst);
        cfg.blockDim = dim3((unsigned)(32 * M < 64 ? 64 : 32 * M));
        cfg.dynamicSmemBytes = (size_t)nact * 128 + 2 * (size_t)sfb_bytes(nact);
        // Up to eight rows its CTAs (8 KB, 256 threads) find room beside the GEMM's CTAs of the
        // call before and wait there.  With more rows they do not (registers): they start when
        // the first SMs become free, and four of them would share one of those SMs and take
        // turns on its issue slots (measured: 5.6 us for the conversion instead of ~1).  Asking
        // for more than half an SM's shared memory puts each on an SM of its own.
        if (M > 8) cfg.dynamicSmemBytes = kActSpread;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = chained ? 1 : 0;
        cudaError_t e = cudaLaunchKernelEx(&cfg, decode_act_kernel, static_cast<const __nv_bfloat16*>(A), lda,
                                           (int)M, nact, ws + kStatusBytes, prm.status, chained ? 0 : 1);
        if (e != cudaSuccess) return MXP_ERR_CUDA;
    }
    cudaError_t e;
    switch (nact) {
        case 16: e = launch_n<16, 0>(plus, f32, prm, p.ctas, L.total, true, stream); break;
        case 32: e = launch_n<32, 0>(plus, f32, prm, p.ctas, L.total, true, stream); break;
        case 48: e = launch_n<48, 0>(plus, f32, prm, p.ctas, L.total, true, stream); break;
        case 64: e = launch_n<64, 0>(plus, f32, prm, p.ctas, L.total, true, stream); break;
        default: e = launch_n<80, 0>(plus, f32, prm, p.ctas, L.total, true, stream); break;
    }
    return e == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

}  // namespace mxp
